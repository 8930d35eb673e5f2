"""The seeded input generators: determinism, shapes, distributions, paging."""
import math

import numpy as np
import torch

from paper_2603_22910_b200 import synth


def test_configs_match_benchmark_shapes():
    assert (synth.C0.D, synth.C0.m, synth.C0.d_in, synth.C0.d_drop) == (512, 256, 768, 256)
    assert (synth.C1.D, synth.C1.m, synth.C1.d_in, synth.C1.d_drop) == (4096, 2048, 6144, 2048)
    assert (synth.C2.D, synth.C2.m, synth.C2.d_in, synth.C2.d_drop) == (1024, 256, 1280, 768)
    assert synth.C3.n_layers == 32 and synth.C3.group_size == 4 and synth.C3.random_pages
    assert [synth.c4_point(p, 4096, 1).d_drop for p in (25, 50, 75)] == [256, 512, 768]
    assert sum(0 if synth.C3.is_anchor(l) else 1 for l in range(32)) == 24


def test_generators_are_deterministic_and_independent():
    w = synth.C0
    a = synth.layer_cache(w, 0, "k", 0)
    b = synth.layer_cache(w, 0, "k", 0)
    assert torch.equal(a, b)
    assert not torch.equal(a, synth.layer_cache(w, 0, "v", 0))
    assert torch.equal(synth.predictor_weights(w, 1, "k"), synth.predictor_weights(w, 1, "k"))
    assert not torch.equal(synth.predictor_weights(w, 1, "k"), synth.predictor_weights(w, 1, "v"))
    # narrower view = prefix of the wider one
    assert torch.equal(synth.layer_cache(w, 1, "k", 0, width=w.m), synth.layer_cache(w, 1, "k", 0)[:, :w.m])


def test_distributions():
    w = synth.C0.replace(context=4096)
    a = synth.layer_cache(w, 0, "k", 0).double()
    c = synth.layer_cache(w, 1, "k", 0).double()
    assert abs(a.mean()) < 0.01 and abs(a.std() - 1) < 0.01
    assert abs(c.std() - 1) < 0.01
    corr = (a * c).mean() / (a.std() * c.std())
    assert abs(corr - w.rho) < 0.01
    W = synth.predictor_weights(w, 1, "k").double()
    bound = math.sqrt(6.0 / (w.d_in + w.d_drop))
    assert W.abs().max() <= bound and W.abs().max() > 0.99 * bound
    assert abs(W.std() - bound / math.sqrt(3)) < 0.01 * bound
    q = synth.queries(w, 1)
    assert q.shape == (1, 8, 64)


def test_block_table_and_paged_pool_round_trip():
    w = synth.C0.replace(batch=3, context=37, random_pages=True)
    n_pages = 16
    tbl = synth.block_table(w, n_pages)
    assert tbl.shape == (3, 3) and len(set(tbl.flatten().tolist())) == 9
    seqs = [synth.layer_cache(w, 1, "k", b, width=w.m) for b in range(3)]
    pool = synth.paged_pool(w, seqs, tbl, n_pages, w.m)
    for b in range(3):
        for t in (0, 15, 16, 36):
            assert torch.equal(pool[tbl[b, t // 16], t % 16], seqs[b][t])
    ident = synth.block_table(w.replace(random_pages=False))
    assert ident.flatten().tolist() == list(range(9))


def test_bf16_bits_view():
    x = torch.tensor([1.0, -2.5, 3.140625], dtype=torch.bfloat16)
    bits = synth.to_numpy_stored(x)
    assert bits.dtype == np.uint16 and bits.tolist() == [0x3F80, 0xC020, 0x4049]
