"""Shared helpers of the GPU parity tests: put a synthetic workload into a library
context, run the oracle on the same stored values, compare."""
from __future__ import annotations

import numpy as np
import torch

from oracle import echokv_oracle as O
from paper_2603_22910_b200 import binding, synth

# tolerances (the benchmark contract): bf16 storage / fp32 accumulate, and the fp32 test mode
TOL = {"bf16": dict(max_abs=2e-2, rel_l2=5e-3), "fp32": dict(max_abs=1e-4, rel_l2=1e-5)}


class Case:
    """One workload resident on the GPU (all layers), plus the host copies the oracle reads."""

    def __init__(self, w: synth.Workload, lens=None, n_pages=None, layers=None, keep_host=True,
                 biases=False, window=None, rope=None):
        """window = (n_sink, n_window): those tokens of every sequence keep all their dims (Section 4.1).
        rope = theta: the cache holds un-rotated keys that are rotated to their positions when read."""
        self.w = w
        self.lens = list(lens) if lens is not None else [w.context] * w.batch
        assert len(self.lens) == w.batch and max(self.lens) <= w.context
        n_pages = n_pages or w.batch * w.pages_per_seq
        self.cfg = binding.config_for(w, n_pages=n_pages)
        self.ctx = binding.Context(self.cfg, zero_pools=False)
        self.table = synth.block_table(w, n_pages)
        self.ctx.set_block_table(self.table)
        self.layers = list(range(w.n_layers)) if layers is None else layers
        self.window = window
        if window:
            self.ctx.set_full_precision_window(*window)
        self.rope = rope
        if rope:
            self.ctx.set_rope(rope)
        self.true_drop = {}  # (layer, kind, b) -> the layer's own dims m..D-1 [len_b, D - m] (window tests)
        self.host = {}       # (layer, kind, b) -> stored-precision tensor [len_b, width]
        self.weights = {}    # layer -> (Wk, Wv, bk, bv) device tensors
        self.host_w = {}
        dev = self.ctx.device
        needed = set(self.layers) | {w.anchor_of(l) for l in self.layers}
        for l in sorted(needed):
            for kind in ("k", "v"):
                # a compressed layer stores m dims of K and V -- or all of K in the "save K" setting
                width = w.D if w.is_anchor(l) else (w.mk if kind == "k" else w.m)
                side_only = width == 0 and bool(window) and not w.is_anchor(l)
                if width == 0 and not side_only:
                    continue
                seqs = []
                for b in range(w.batch):
                    x = synth.layer_cache(w, l, kind, b, width=max(width, 1))[: self.lens[b]][:, :width]
                    seqs.append(x)
                    if keep_host and width:
                        self.host[(l, kind, b)] = x
                # all tokens but the last go in directly; the last one is appended by the library
                if width:
                    pool = synth.paged_pool(w, [s[:-1] for s in seqs], self.table, n_pages, width)
                    (self.ctx.k_pools if kind == "k" else self.ctx.v_pools)[l].copy_(pool)
                newest = torch.zeros((w.batch, w.D), dtype=synth.torch_dtype(w))
                for b in range(w.batch):
                    newest[b, :width] = seqs[b][-1]
                    if width < w.D:
                        newest[b, width:] = 777.0   # must never reach the cache
                if window and not w.is_anchor(l) and w.D > w.m:
                    # the sink / window tokens' own dims m..D-1: all but the newest are placed in the side
                    # buffers here, the newest goes through the library's append
                    n_sink, n_window = window
                    side = (self.ctx.k_side if kind == "k" else self.ctx.v_side)[l]
                    for b in range(w.batch):
                        L = self.lens[b]
                        full = synth.layer_cache(w, l, kind, b, width=w.D)[:L]
                        self.true_drop[(l, kind, b)] = full[:, w.m:]
                        newest[b, w.m:] = full[-1, w.m:]
                        for t in range(L - 1):
                            if t < n_sink:
                                side[b, t] = full[t, w.m:].to(dev)
                            if n_window and t >= L - 1 - n_window:      # still inside the ring after the append
                                side[b, n_sink + t % n_window] = full[t, w.m:].to(dev)
                self.host[(l, kind, "new")] = newest
            if not w.is_anchor(l):
                Wk = synth.predictor_weights(w, l, "k")
                Wv = synth.predictor_weights(w, l, "v")
                bk = bv = None
                if biases:
                    bk = (synth.normal((w.d_drop,), w.seed, 90, l) * 0.1).to(synth.torch_dtype(w))
                    bv = (synth.normal((w.d_drop,), w.seed, 91, l) * 0.1).to(synth.torch_dtype(w))
                self.host_w[l] = (Wk, Wv, bk, bv)
                devw = tuple(None if t is None else t.to(dev) for t in (Wk, Wv, bk, bv))
                if w.save_k:
                    devw = (None, devw[1], None, devw[3])     # keys kept whole: the library takes no K predictor
                self.weights[l] = devw
                self.ctx.set_weights(l, *devw)
        self.seq_lens = torch.tensor(self.lens, dtype=torch.int32, device=dev)
        self.positions = self.seq_lens - 1
        for l in sorted(needed):
            if (l, "k", "new") in self.host:
                v_new = self.host.get((l, "v", "new"))
                if v_new is None:        # nothing of V is stored on this layer: whatever is passed must be ignored
                    v_new = torch.full((w.batch, w.D), 777.0, dtype=synth.torch_dtype(w))
                self.ctx.append_kv(l, self.host[(l, "k", "new")].to(dev), v_new.to(dev), self.positions)
        self.q = {l: synth.queries(w, l) for l in self.layers}

    def run(self, layer, full=False):
        q = self.q[layer].to(self.ctx.device)
        fn = self.ctx.full_attention if full else self.ctx.decode_attention
        out = fn(layer, q, self.seq_lens)
        torch.cuda.synchronize()
        return out.cpu().numpy().astype(np.float64)

    def _stored(self, layer, kind, b):
        return O.widen(synth.to_numpy_stored(self.host[(layer, kind, b)]))

    def oracle(self, layer, batch_indices=None, query_heads=None):
        """Oracle output [B, H_q, d] (or, with query_heads, {(b, h): [d]})."""
        w = self.w
        bs = range(w.batch) if batch_indices is None else batch_indices
        qn = O.widen(synth.to_numpy_stored(self.q[layer]))
        res = {} if query_heads is not None else np.zeros((w.batch, w.n_q_heads, w.head_dim))
        for b in bs:
            if w.is_anchor(layer):
                kk, vv = self._stored(layer, "k", b), self._stored(layer, "v", b)
                if query_heads is None:
                    res[b] = O.full_attention(qn[b], kk, vv, w.n_kv_heads, rope_theta=self.rope)
                else:
                    full = O.full_attention(qn[b], kk, vv, w.n_kv_heads, rope_theta=self.rope)
                    for h in query_heads:
                        res[(b, h)] = full[h]
                continue
            a = w.anchor_of(layer)
            kg, vg = self._stored(a, "k", b), self._stored(a, "v", b)
            L = kg.shape[0]
            k_true = self._stored(layer, "k", b) if w.save_k else None      # keys kept whole
            kl = (k_true[:, :w.m] if w.save_k else self._stored(layer, "k", b)) if w.m else np.zeros((L, 0))
            vl = self._stored(layer, "v", b) if w.m else np.zeros((L, 0))
            Wk, Wv, bk, bv = (None if t is None else O.widen(synth.to_numpy_stored(t))
                              for t in self.host_w[layer])
            if self.window and w.D > w.m:
                kt = O.widen(synth.to_numpy_stored(self.true_drop[(layer, "k", b)]))
                vt = O.widen(synth.to_numpy_stored(self.true_drop[(layer, "v", b)]))
                assert query_heads is None
                res[b] = O.decode_attention_windowed(qn[b], kg, vg, kl, vl, Wk, Wv, w.n_kv_heads, kt, vt,
                                                     self.window[0], self.window[1], bk=bk, bv=bv,
                                                     rope_theta=self.rope, k_true=k_true)
            elif query_heads is None:
                res[b] = O.decode_attention(qn[b], kg, vg, kl, vl, Wk, Wv, w.n_kv_heads, bk=bk, bv=bv,
                                            rope_theta=self.rope, k_true=k_true)
            else:
                per = O.decode_attention_query_heads(qn[b], kg, vg, kl, vl, Wk, Wv, w.n_kv_heads, query_heads,
                                                     rope_theta=self.rope)
                for h, v in per.items():
                    res[(b, h)] = v
        return res

    def recent_rows(self, layer, n_q):
        """Full-width K and V rows of the last n_q + n_window - 1 tokens of every sequence, [B][n][D] on the
        device (rows of positions before the sequence's start are zero): what the prefill-shaped call takes
        when a window is set."""
        w = self.w
        n = n_q + self.window[1] - 1
        outs = []
        for kind in ("k", "v"):
            rows = torch.zeros((w.batch, n, w.D), dtype=synth.torch_dtype(w))
            for b in range(w.batch):
                full = synth.layer_cache(w, layer, kind, b, width=w.D)[: self.lens[b]]
                take = min(n, full.shape[0])
                rows[b, n - take:] = full[full.shape[0] - take:]
            outs.append(rows.to(self.ctx.device))
        return outs

    def close(self):
        self.ctx.close()


def errors(out: np.ndarray, ref: np.ndarray):
    out = np.asarray(out, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    max_abs = float(np.max(np.abs(out - ref))) if out.size else 0.0
    rel_l2 = float(np.linalg.norm(out - ref) / max(np.linalg.norm(ref), 1e-300))
    return max_abs, rel_l2


def assert_parity(out, ref, dtype: str, what: str = ""):
    max_abs, rel_l2 = errors(out, ref)
    tol = TOL[dtype]
    assert np.all(np.isfinite(out)), "non-finite output " + what
    assert max_abs <= tol["max_abs"] and rel_l2 <= tol["rel_l2"], \
        "%s: max_abs %.3e (tol %.1e), rel_l2 %.3e (tol %.1e)" % (what, max_abs, tol["max_abs"], rel_l2, tol["rel_l2"])
    return max_abs, rel_l2
