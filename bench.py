#!/usr/bin/env python
"""Benchmark of the EchoKV decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]
                    [--workload c1|c2|c3|c4] [--mode compressed|full] [--sweep] ...

One "step" = one pass of the whole hot path over one batch of synthetic input.  For the
single-layer workloads (c1; c2; a point of the c4 sweep) that is: append the new token to the
anchor layer and to the compressed layer (which keeps only the retained dims), then decode
attention on the compressed layer -- retained heads from the cache, dropped heads reconstructed
on chip -- including the split-K merge.  For c3 it is the whole 32-layer decode step: per layer an
append and the layer's attention (full-cache on the 8 anchor layers, reconstruct-then-attend on the
24 compressed ones).  --mode full times the uncompressed path instead.

Without --workload the run is the whole record: the headline is the largest single-GPU
configuration (c3: 32 layers, 16-token pages in a random order), followed by a `sustained` leg
(the same step repeated for at least two seconds, with the clocks sampled throughout) and a
`configs` object with one sub-record per benchmark configuration (c1, c2, c3 and three points of
the c4 sweep), each with its step time, its end-to-end time, the dominant kernel's time and its
fraction of both measured tensor peaks, a parity sample against the CPU oracle and the
uncompressed step at the same shape.  With --workload only that workload is measured.
`--workload c4 --sweep` walks the whole sweep (ratio x context x batch), one sub-record per point.

`value` is decode tokens per second (sequences advanced per second) with the caches resident
in HBM; `e2e` is the same step driven from pinned host buffers through
echokv_layer_step_host.  With N > 1 every rank runs an independent replica of the batch (the
path has no exchange step): weak scaling, no collective on the data path.

--impl reference times the CPU oracle (numpy, fp64) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"

HEADLINE = "c3"
# the sub-records of the default run: every benchmark configuration that fits a short run
SUITE = [
    ("c1", dict(workload="c1")),
    ("c2", dict(workload="c2")),
    ("c3", dict(workload="c3")),
    ("c4_75pct_B8_L65536", dict(workload="c4", ratio=75, batch=8, context=65536)),
    ("c4_75pct_B2_L131072", dict(workload="c4", ratio=75, batch=2, context=131072)),
    ("c4_25pct_B8_L16384", dict(workload="c4", ratio=25, batch=8, context=16384)),
]

# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum) from
# the ncu captures summarised under profiles/; None until a capture of that workload exists.
NCU_TRAFFIC_BYTES = {
    # B = 2 captures of the same layer shape, scaled by the tokens of a full launch (traffic grows with the rows read)
    "c1": 4 * 620.7e6,        # recon_quad_kernel, pages in order: B = 2 capture x 4
    "c3": 4 * 620.5e6,        # recon_quad_kernel per launch (one compressed layer; 65 536 tokens as C1), 16-token
                              # pages in a random order: B = 2, L = 8192 capture x 4
    "c2": 8 * 348.6e6,        # recon_pair_kernel: B = 2 capture x 8
    "c1_full": 4 * 272.1e6,   # attn_stored_mma_kernel: B = 2 capture x 4
    "c2_full": 8 * 273.9e6,   # attn_stored_mma_kernel: B = 2 capture x 8
    "c1_absorbed": 4 * 418.7e6,   # absorb_scores_kernel + absorb_pv_kernel (one launch each): B = 2 capture x 4
    "c2_absorbed": 8 * 354.7e6,   # the same: B = 2 capture x 8
}

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def traffic_of(args, key):
    """The stored ncu figure, only for the exact workload and kernel it was taken on."""
    if args.batch or args.context or args.page_tokens or args.random_pages:
        return None
    if (args.rope or args.window or args.retained_dims or args.save_k or args.decode_path is not None
            or args.stored_path is not None):
        return None          # another kernel (instantiation) than the captured one
    return NCU_TRAFFIC_BYTES.get(key)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload_by_name(name, batch=0, context=0, page_tokens=0, random_pages=False, ratio=75, retained_dims=0,
                     save_k=False):
    from paper_2603_22910_b200 import synth
    if save_k:    # keys kept whole on compressed layers, only the values predicted (the paper's "save K" setting)
        w = workload_by_name(name, batch, context, page_tokens, random_pages, ratio, retained_dims)
        return w.replace(save_k=True, name=w.name + "_saveK")
    if name == "c4":
        w = synth.c4_point(ratio, context or 16384, batch or 8)
        if retained_dims:   # the paper's own settings, e.g. m = 64: half of the first head
            w = w.replace(n_retained_dims=retained_dims, n_retained_heads=retained_dims // w.head_dim,
                          name="c4_m%d_L%d_B%d" % (retained_dims, w.context, w.batch))
        if page_tokens:
            w = w.replace(page_tokens=page_tokens, name=w.name + "_P%d" % page_tokens)
        if random_pages:
            w = w.replace(random_pages=True, name=w.name + "_randpages")
        return w
    w = {"c1": synth.C1, "c2": synth.C2, "c3": synth.C3}[name]
    if page_tokens:
        w = w.replace(page_tokens=page_tokens, name=w.name + "_P%d" % page_tokens)
    if random_pages:
        w = w.replace(random_pages=True, name=w.name + "_randpages")
    if batch:
        w = w.replace(batch=batch, name=w.name + "_B%d" % batch)
    if context:
        w = w.replace(context=context, name=w.name + "_L%d" % context)
    return w


def workload_of_args(args):
    return workload_by_name(args.workload or HEADLINE, args.batch, args.context, args.page_tokens, args.random_pages,
                            args.ratio, args.retained_dims, args.save_k)


def algorithmic_work(w):
    """Per launch of the fused kernel (one compressed layer): FLOPs of Eq. 3 (both predictors) plus
    Eq. 7 on the dropped heads, and the bytes the method must move (predictor inputs once,
    predictors once)."""
    tokens = w.batch * w.context
    g = w.n_q_heads // w.n_kv_heads
    n_drop_q = (w.n_kv_heads - w.m // w.head_dim) * g
    flops = tokens * (4.0 * w.d_in * w.d_drop + 4.0 * n_drop_q * w.head_dim)
    elem = 2 if w.dtype == "bf16" else 4
    bytes_ = tokens * 2.0 * w.d_in * elem + 2.0 * w.d_in * w.d_drop * elem
    return flops, bytes_


class ClockSampler(threading.Thread):
    """Samples SM clock, power and throttle reasons through NVML (read-only) while a timed region runs."""

    def __init__(self, index, period_s=0.002):
        super().__init__(daemon=True)
        self.index = index
        self.period_s = period_s
        self.samples, self.power, self.reasons = [], [], set()
        self.max_mhz = None
        self._stop_evt = threading.Event()
        self.error = None

    def run(self):
        try:
            import pynvml as nv
            nv.nvmlInit()
            h = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(h, nv.NVML_CLOCK_SM)
            names = {
                getattr(nv, "nvmlClocksEventReasonGpuIdle", 0x1): "gpu_idle",
                getattr(nv, "nvmlClocksEventReasonApplicationsClocksSetting", 0x2): "applications_clocks_setting",
                getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
                getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
                getattr(nv, "nvmlClocksEventReasonSyncBoost", 0x10): "sync_boost",
                getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
                getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake_slowdown",
            }
            while not self._stop_evt.is_set():
                self.samples.append(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM))
                try:
                    self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
                except Exception:
                    pass
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
                time.sleep(self.period_s)
        except Exception as e:  # NVML missing: report it rather than guess
            self.error = repr(e)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        s = sorted(self.samples)
        med = s[len(s) // 2] if s else None
        out = {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s)}
        if s:
            out["sm_mhz_min"] = s[0]
        if self.power:
            out["power_w_max"] = max(self.power)
        if self.error:
            out["error"] = self.error
        return out


def physical_gpu_index(local_index):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        parts = [p.strip() for p in vis.split(",") if p.strip()]
        if local_index < len(parts) and parts[local_index].isdigit():
            return int(parts[local_index])
    return local_index


# --------------------------------------------------------------------------------------------
# Workload state on the GPU
# --------------------------------------------------------------------------------------------
class State:
    """A workload resident on one GPU: pools filled through the block table from the seeded
    generators (drawn on the device: the largest workloads do not fit host memory), predictors,
    one decode query per layer, and the newest token of every layer (re-appended by each step)."""

    def __init__(self, w, local_rank, layers, window=None):
        import torch
        from paper_2603_22910_b200 import binding, synth
        self.w, self.layers = w, layers
        self.window = window if (window and w.D > w.m) else None
        self.rope = None
        self.dev = dev = torch.device("cuda", local_rank)
        self.ctx = ctx = binding.Context(binding.config_for(w, device=local_rank))
        if self.window:
            ctx.set_full_precision_window(*self.window)
        self.true_rows = {}   # (layer, kind, b) -> (token indices, their dims m..D-1): sink and window tokens
        self.table = synth.block_table(w)
        ctx.set_block_table(self.table)
        t0 = time.perf_counter()
        needed = sorted(set(layers) | {w.anchor_of(l) for l in layers})
        tdt = synth.torch_dtype(w)
        self.new_dev, self.new_host, self.q_dev, self.q_host = {}, {}, {}, {}
        for l in needed:
            for kind, pools in (("k", ctx.k_pools), ("v", ctx.v_pools)):
                width = w.D if w.is_anchor(l) else (w.mk if kind == "k" else w.m)
                side = self.window and not w.is_anchor(l) and not (w.save_k and kind == "k")
                newest = torch.zeros((w.batch, w.D), dtype=tdt, device=dev)
                for b in range(w.batch):
                    if width == 0 and not side:
                        continue
                    ids = self.table[b].long().to(dev)
                    x = synth.layer_cache(w, l, kind, b, width=w.D if side else width, device=dev)
                    if side:
                        # sink and recent-window tokens keep their dims m..D-1 in the side buffers
                        n_sink, n_window = self.window
                        L = w.context
                        toks = [t for t in range(L) if t < n_sink or t >= L - n_window]
                        tt = torch.tensor(toks, device=dev)
                        rows = x[tt, w.m:]
                        buf = (ctx.k_side if kind == "k" else ctx.v_side)[l]
                        slots = torch.tensor([t if t < n_sink else n_sink + t % n_window for t in toks], device=dev)
                        buf[b, slots] = rows          # (a sink token inside the window: same values twice)
                        self.true_rows[(l, kind, b)] = (toks, rows.cpu())
                        newest_full = x[w.context - 1].clone()
                        x = x[:, :width].contiguous()
                    else:
                        newest_full = None
                    if width:
                        pad = w.pages_per_seq * w.page_tokens - w.context
                        if pad:
                            x = torch.cat([x, torch.zeros((pad, width), dtype=tdt, device=dev)])
                        pools[l][ids] = x.reshape(w.pages_per_seq, w.page_tokens, width)
                        newest[b, :width] = x[w.context - 1]
                    if newest_full is not None:
                        newest[b] = newest_full        # the step re-appends the newest token, all its dims
                    del x
                self.new_dev[(l, kind)] = newest
                self.new_host[(l, kind)] = newest.cpu().pin_memory()
            if not w.is_anchor(l):
                Wk = synth.predictor_weights(w, l, "k", device=dev)
                Wv = synth.predictor_weights(w, l, "v", device=dev)
                ctx.set_weights(l, None if w.save_k else Wk, Wv)
            self.q_dev[l] = synth.queries(w, l, device=dev)
            self.q_host[l] = self.q_dev[l].cpu().pin_memory()
        self.lens_host = torch.full((w.batch,), w.context, dtype=torch.int32).pin_memory()
        self.lens = self.lens_host.to(dev)
        self.positions = self.lens - 1
        shape = (w.batch, w.n_q_heads, w.head_dim)
        self.out = {l: torch.empty(shape, dtype=torch.float32, device=dev) for l in layers}
        self.out_host = {l: torch.empty(shape, dtype=torch.float32).pin_memory() for l in layers}
        torch.cuda.synchronize()
        self.gen_s = time.perf_counter() - t0

    def stored_sequence(self, layer, kind, b):
        """Stored values [L, width] of one sequence, gathered back from the pool (oracle input)."""
        pools = self.ctx.k_pools if kind == "k" else self.ctx.v_pools
        if pools[layer] is None:
            import torch
            return torch.zeros((self.w.context, 0), dtype=self.ctx.tdtype)
        ids = self.table[b].long().to(self.dev)
        x = pools[layer][ids].reshape(-1, pools[layer].shape[-1])[: self.w.context]
        return x.cpu()

    def oracle_inputs(self, layer, b):
        """Widened (float64) oracle inputs of sequence b at `layer`, from what the GPU holds."""
        from oracle import echokv_oracle as O
        from paper_2603_22910_b200 import synth
        w = self.w
        st = synth.to_numpy_stored
        a = w.anchor_of(layer)
        q = O.widen(st(self.q_host[layer]))[b]
        kg = O.widen(st(self.stored_sequence(a, "k", b)))
        vg = O.widen(st(self.stored_sequence(a, "v", b)))
        if w.is_anchor(layer):
            return q, kg, vg
        kl = O.widen(st(self.stored_sequence(layer, "k", b)))[:, :w.m]
        vl = O.widen(st(self.stored_sequence(layer, "v", b)))
        Wk, Wv = (None if t is None else O.widen(st(t)) for t in self.ctx._weights[layer][:2])
        return q, kg, vg, kl, vl, Wk, Wv

    def true_keys(self, layer, b):
        """The layer's whole keys [L, D] where it keeps them ("save K"), else None."""
        from oracle import echokv_oracle as O
        from paper_2603_22910_b200 import synth
        if not self.w.save_k or self.w.is_anchor(layer):
            return None
        return O.widen(synth.to_numpy_stored(self.stored_sequence(layer, "k", b)))

    def true_dropped(self, layer, kind, b):
        """[L, D - m] with the sink / window tokens' own dims m..D-1 (NaN elsewhere: never read)."""
        import numpy as np
        from oracle import echokv_oracle as O
        from paper_2603_22910_b200 import synth
        out = np.full((self.w.context, self.w.D - self.w.m), np.nan)
        if (layer, kind, b) in self.true_rows:
            toks, rows = self.true_rows[(layer, kind, b)]
            out[toks] = O.widen(synth.to_numpy_stored(rows))
        return out


def plan_layers(w, mode):
    """(layers resident on the GPU, [(layer, attend?)] of one step)."""
    if mode == "full":
        return [0], [(0, True)]
    if w.n_layers > 2:                     # the whole multi-layer decode step
        return list(range(w.n_layers)), [(l, True) for l in range(w.n_layers)]
    return [0, 1], [(0, False), (1, True)]  # the anchor only receives its token; layer 1 attends


# --------------------------------------------------------------------------------------------
# CPU oracle legs
# --------------------------------------------------------------------------------------------
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_layer(inputs, w, state=None, layer=None, b=None):
    from oracle import echokv_oracle as O
    rope = getattr(state, "rope", None) or None
    if len(inputs) == 3:
        return O.full_attention(inputs[0], inputs[1], inputs[2], w.n_kv_heads, rope_theta=rope)
    k_true = state.true_keys(layer, b) if state is not None else None
    if state is not None and state.window:
        return O.decode_attention_windowed(*inputs, w.n_kv_heads, state.true_dropped(layer, "k", b),
                                           state.true_dropped(layer, "v", b), state.window[0], state.window[1],
                                           rope_theta=rope, k_true=k_true)
    return O.decode_attention(*inputs, n_kv_heads=w.n_kv_heads, rope_theta=rope, k_true=k_true)


def oracle_heads(state, layer, b, heads, inputs=None):
    """Oracle outputs {h: [d]} of a few query heads of (layer, sequence b): heads are independent in Eq. 7
    and a predicted head needs only its own rows of W in Eq. 3."""
    from oracle import echokv_oracle as O
    w = state.w
    rope = state.rope or None
    inputs = state.oracle_inputs(layer, b) if inputs is None else inputs
    if len(inputs) == 3:                # a stored (anchor / uncompressed) layer: only the head's own dims
        q, kg, vg = inputs
        d, g = w.head_dim, w.n_q_heads // w.n_kv_heads
        out = {}
        for h in heads:
            kv = h // g
            out[h] = O.attention(q[h:h + 1], kg[:, None, kv * d:(kv + 1) * d], vg[:, None, kv * d:(kv + 1) * d],
                                 rope_theta=rope)[0]
        return out
    kw = {}
    if state.window:
        kw = dict(k_true_drop=state.true_dropped(layer, "k", b), v_true_drop=state.true_dropped(layer, "v", b),
                  n_sink=state.window[0], n_window=state.window[1])
    k_true = state.true_keys(layer, b)
    if k_true is not None:
        kw["k_true"] = k_true
    return O.decode_attention_query_heads(*inputs, n_kv_heads=w.n_kv_heads, query_heads=list(heads), rope_theta=rope,
                                          **kw)


def stratified_picks(w, attend_layers, n_outputs, seed=7, max_combos=16):
    """[(layer, sequence, [query heads])] covering, between them: every sequence of the batch, the first, a
    middle and the last compressed layer and the first and last anchor layer of the step, and every KV head
    (dropped heads first, so every pair of dropped heads a fused-kernel work item handles is met)."""
    import numpy as np
    rng = np.random.default_rng(seed)
    g = w.n_q_heads // w.n_kv_heads
    comp = [l for l in attend_layers if not w.is_anchor(l) and w.d_drop > 0]
    anch = [l for l in attend_layers if l not in comp]
    layers = []
    if comp:
        layers += sorted({comp[0], comp[len(comp) // 2], comp[-1]})
    if anch:
        layers += sorted({anch[0], anch[-1]})
    n_combos = min(max(w.batch, len(layers)), max_combos, n_outputs)
    per = int(math.ceil(n_outputs / float(n_combos)))
    first_drop = w.m // w.head_dim            # (a partly retained head is predicted in part: counts as dropped)
    picks, walk = [], 0
    for k in range(n_combos):
        l, b = layers[k % len(layers)], k % w.batch
        if w.is_anchor(l) or w.d_drop == 0:
            kv_order = list(range(w.n_kv_heads))
        else:
            kv_order = list(range(first_drop, w.n_kv_heads)) + list(range(first_drop))
        heads = []
        for _ in range(per):
            kv = kv_order[walk % len(kv_order)]
            walk += 1
            h = kv * g + int(rng.integers(g))
            if h not in heads:
                heads.append(h)
        picks.append((l, b, heads))
    return picks


def parity_sample(state, picks):
    """Element-wise comparison of sampled GPU outputs (state.out, as the last step left them) with the oracle."""
    import numpy as np
    worst = num = den = 0.0
    n = 0
    for l, b, heads in picks:
        ref = oracle_heads(state, l, b, heads)
        for h in heads:
            got = state.out[l][b, h].cpu().numpy().astype(np.float64)
            if not np.all(np.isfinite(got)):
                return {"outputs": n, "max_abs": float("inf"), "rel_l2": float("inf")}
            worst = max(worst, float(np.max(np.abs(got - ref[h]))))
            num += float(np.sum((got - ref[h]) ** 2))
            den += float(np.sum(ref[h] ** 2))
            n += 1
    return {"outputs": n, "combos": [(l, b, len(hs)) for l, b, hs in picks], "max_abs": worst,
            "rel_l2": (num / max(den, 1e-300)) ** 0.5}


def time_oracle(state, step_layers, budget_s):
    """The oracle as it stands on a bounded sample of the workload.  Returns (tokens/s of the
    oracle scaled to the whole step, sample description, {(layer, b): oracle output})."""
    w = state.w
    attend = [l for l, a in step_layers if a]
    outs, elapsed = {}, 0.0
    if len(attend) == 1:
        # whole sequences of the batch, all heads, all tokens, until the budget is used
        layer = attend[0]
        for b in range(min(w.batch, 4)):
            inputs = state.oracle_inputs(layer, b)
            t0 = time.perf_counter()
            outs[(layer, b)] = oracle_layer(inputs, w, state, layer, b)
            elapsed += time.perf_counter() - t0
            if elapsed >= budget_s:
                break
        n_seq = len(outs)
        return n_seq / elapsed, ("%d of %d sequences of the batch, all heads, all %d tokens (%.1f s)"
                                 % (n_seq, w.batch, w.context, elapsed)), outs
    # multi-layer step: whole sequences through the first anchor layer and the first compressed layer (every
    # anchor layer costs the same, every compressed layer costs the same), scaled to the layer counts
    anchors = [l for l in attend if w.is_anchor(l)]
    comps = [l for l in attend if not w.is_anchor(l)]
    t_kind = {"a": 0.0, "c": 0.0}
    n_seq = 0
    for b in range(w.batch):
        for kind, ls in (("a", anchors), ("c", comps)):
            if not ls:
                continue
            inputs = state.oracle_inputs(ls[0], b)
            t0 = time.perf_counter()
            outs[(ls[0], b)] = oracle_layer(inputs, w, state, ls[0], b)
            t_kind[kind] += time.perf_counter() - t0
        n_seq += 1
        if t_kind["a"] + t_kind["c"] >= budget_s:
            break
    t_seq = (t_kind["a"] * len(anchors) + t_kind["c"] * len(comps)) / n_seq     # one sequence, all layers
    return 1.0 / t_seq, ("%d of %d sequences through layer %d (anchor) and layer %d (compressed), all heads, all %d "
                         "tokens (%.1f s); scaled to %d anchor + %d compressed layers"
                         % (n_seq, w.batch, anchors[0] if anchors else -1, comps[0] if comps else -1, w.context,
                            t_kind["a"] + t_kind["c"], len(anchors), len(comps))), outs


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import echokv_oracle as O
    from paper_2603_22910_b200 import synth
    w = workload_of_args(args)
    st = synth.to_numpy_stored
    full = args.mode == "full"
    rope = args.rope or None
    # One step evaluates sequence 0 of the batch, all heads, all tokens, for one layer (single-layer workloads)
    # or for the first anchor layer and the first compressed layer (the 32-layer workload: every anchor layer
    # costs the same and every compressed layer costs the same).  ms_per_step is the time of that sample as
    # measured; only `value` is scaled to the batch and the layer counts.
    multi = w.n_layers > 2 and not full
    layers = [0, 1] if multi else [0 if full else 1]
    inputs, k_true = {}, {}
    for l in layers:
        a = w.anchor_of(l)
        q = O.widen(st(synth.queries(w, l)))[0]
        kg = O.widen(st(synth.layer_cache(w, a, "k", 0)))
        vg = O.widen(st(synth.layer_cache(w, a, "v", 0)))
        if full or w.is_anchor(l):
            inputs[l] = (q, kg, vg)
        else:
            k_true[l] = O.widen(st(synth.layer_cache(w, l, "k", 0, width=w.D))) if w.save_k else None
            inputs[l] = (q, kg, vg,
                         O.widen(st(synth.layer_cache(w, l, "k", 0, width=w.m))),
                         O.widen(st(synth.layer_cache(w, l, "v", 0, width=w.m))),
                         O.widen(st(synth.predictor_weights(w, l, "k"))),
                         O.widen(st(synth.predictor_weights(w, l, "v"))))

    def run():
        per_layer = {}
        for l in layers:
            x = inputs[l]
            t0 = time.perf_counter()
            if len(x) == 3:
                O.full_attention(x[0], x[1], x[2], w.n_kv_heads, rope_theta=rope)
            else:
                O.decode_attention(*x, n_kv_heads=w.n_kv_heads, rope_theta=rope, k_true=k_true[l])
            per_layer[l] = time.perf_counter() - t0
        return per_layer

    times, per = [], {l: [] for l in layers}
    for i in range(args.steps + args.warmup):
        t0 = time.perf_counter()
        pl = run()
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
            for l in layers:
                per[l].append(pl[l])
    t_step = sum(times) / len(times)
    if multi:
        n_anchor = (w.n_layers + w.group_size - 1) // w.group_size
        t_seq = (sum(per[0]) / len(per[0])) * n_anchor + (sum(per[1]) / len(per[1])) * (w.n_layers - n_anchor)
        scaled = "value scaled to %d anchor + %d compressed layers" % (n_anchor, w.n_layers - n_anchor)
    else:
        t_seq = t_step
        scaled = "value = sequences per second of this sample"
    value = 1.0 / t_seq                  # sequences advanced per second = decode tokens per second
    sample = ("each step: sequence 0 of %d, %s, all heads, all %d tokens; ms_per_step is that sample as measured; %s"
              % (w.batch, "layer 0 (anchor) and layer 1 (compressed)" if multi else "one layer", w.context, scaled))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_step * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w, full),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def run_prefill(args):
    """--prefill-queries N: the prefill-shaped call on the compressed layer (N causal queries per sequence at the end
    of the cached context), timed on the device; an extra measurement beside the decode benchmark, one JSON line."""
    import numpy as np
    import torch
    from paper_2603_22910_b200 import binding, synth
    from oracle import echokv_oracle as O
    w = workload_of_args(args)
    n_q = args.prefill_queries
    window = parse_window(args)
    st = State(w, 0, [0, 1], window)
    ctx, dev = st.ctx, st.dev
    if args.rope:
        ctx.set_rope(args.rope)
    st.rope = args.rope
    q = synth.normal((w.batch, n_q, w.n_q_heads, w.head_dim), w.seed, 77, 1, device=dev).to(torch.bfloat16)
    out = torch.empty(q.shape, dtype=torch.float32, device=dev)
    recent = {}
    if st.window:
        # whole K / V rows of the chunk and the n_window - 1 tokens before it (what a caller has at hand while it
        # prefills in chunks): the call reads every query's own window from them
        n_rows = n_q + st.window[1] - 1
        for kind in ("k", "v"):
            recent[kind + "_recent"] = torch.stack([synth.layer_cache(w, 1, kind, b, width=w.D, device=dev)[-n_rows:]
                                                    for b in range(w.batch)]).contiguous()
    for _ in range(max(3, args.warmup)):
        ctx.prefill_attention(1, q, st.lens, out=out, **recent)
    torch.cuda.synchronize()
    ctx.set_kernel_timing(True)
    ctx.read_kernel_timing_by_kind()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ctx.prefill_attention(1, q, st.lens, out=out, **recent)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    recon_ms, recon_n = ctx.read_kernel_timing_by_kind()["recon"]
    assert ctx.device_status() == binding.ECHOKV_OK
    peaks, peaks_kind = load_peaks()
    tokens = float(w.batch) * w.context
    recon_flops = tokens * 4.0 * w.d_in * w.d_drop
    k_ms = recon_ms / max(recon_n, 1)
    peak_tf = float(peaks["bf16_tflops"])
    # causal attention: query i sees L - n_q + i + 1 keys; 4 d FLOP per (query, key, head)
    seen = n_q * (w.context - n_q) + n_q * (n_q + 1) / 2.0
    attn_flops = w.batch * w.n_q_heads * seen * 4.0 * w.head_dim
    # parity on the last 16 queries of sequence 0 (they see the whole cache)
    n_chk = min(16, n_q)
    inputs = st.oracle_inputs(1, 0)
    q_chk = O.widen(synth.to_numpy_stored(q[0, -n_chk:].cpu()))
    kw = {}
    if st.window:
        # the queries' own windows reach back n_window - 1 tokens before the chunk: their true dims come from the rows
        # handed to the call (the sink tokens' from what the side buffers hold)
        true = {}
        for kind in ("k", "v"):
            t = st.true_dropped(1, kind, 0)
            rows = recent[kind + "_recent"][0].cpu()
            t[w.context - rows.shape[0]:] = O.widen(synth.to_numpy_stored(rows))[:, w.m:]
            true[kind] = t
        kw = dict(k_true_drop=true["k"], v_true_drop=true["v"], n_sink=st.window[0], n_window=st.window[1])
    ref = O.prefill_attention(q_chk, *inputs[1:], n_kv_heads=w.n_kv_heads, rope_theta=args.rope or None, **kw)
    got = out[0, -n_chk:].cpu().numpy().astype(np.float64)
    line = {
        "metric": "prefill_query_tokens_per_s", "value": w.batch * n_q / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "%s, prefill-shaped: %d causal queries per sequence over B=%d L=%d" %
                               (w.name, n_q, w.batch, w.context), "parallelism": "one GPU"},
        "roofline": {"bound": "tensor", "achieved": recon_flops / (k_ms * 1e-3) / 1e12, "peak": peak_tf,
                     "unit": "TFLOP/s", "frac": recon_flops / (k_ms * 1e-3) / 1e12 / peak_tf, "traffic": None,
                     "kernel": "recon_pair_kernel (rows to memory), K pass + V pass", "kernel_ms": k_ms,
                     "share_of_step": k_ms / ms, "peak_source": "%s (cuBLAS bf16 GEMM, burst)" % peaks_kind},
        "attention": {"kernel": "prefill_attn_ws_kernel (tcgen05, warp-specialised) + gather_rows_kernel x 2",
                      "ms": ms - k_ms, "tflops": attn_flops / ((ms - k_ms) * 1e-3) / 1e12},
        "parity_vs_oracle": {"rows": "last %d queries of sequence 0" % n_chk,
                             "max_abs": float(np.max(np.abs(got - ref))),
                             "rel_l2": float(np.linalg.norm(got - ref) / np.linalg.norm(ref))},
        "rope_theta": args.rope or None,
        "full_precision_tokens": {"sink": window[0], "window": window[1]} if window else None,
    }
    print(json.dumps(line))
    ctx.close()
    return 0


def workload_config(w, full=False):
    elem = 2 if w.dtype == "bf16" else 4
    pages = "%d-token pages%s" % (w.page_tokens, " in a random order" if w.random_pages else "")
    if full:
        what = ("%s, uncompressed: B=%d L=%d H_q=%d H_kv=%d d=%d, %s, %s, full-cache attention on the "
                "anchor layer" % (w.name, w.batch, w.context, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype, pages))
        gb = w.batch * w.context * 2 * w.D * elem / 1e9
    elif w.n_layers > 2:
        n_anchor = (w.n_layers + w.group_size - 1) // w.group_size
        what = ("%s: %d layers (S=%d: %d anchor + %d compressed), B=%d L=%d H_q=%d H_kv=%d d=%d m=%d "
                "(D_in=%d -> D_drop=%d), %s, %s" % (w.name, w.n_layers, w.group_size, n_anchor, w.n_layers - n_anchor,
                                                   w.batch, w.context, w.n_q_heads, w.n_kv_heads, w.head_dim,
                                                   w.m, w.d_in, w.d_drop, w.dtype, pages))
        gb = w.batch * w.context * 2 * elem * (n_anchor * w.D + (w.n_layers - n_anchor) * w.d_in) / 1e9
    else:
        what = ("%s: B=%d L=%d H_q=%d H_kv=%d d=%d m=%d (D_in=%d -> D_drop=%d), %s, %s, "
                "anchor + compressed layer" % (w.name, w.batch, w.context, w.n_q_heads, w.n_kv_heads, w.head_dim,
                                               w.m, w.d_in, w.d_drop, w.dtype, pages))
        gb = w.batch * w.context * 2 * w.d_in * elem / 1e9
    return {"workload": what, "global_batch": w.batch, "context": w.context,
            "l2": "inputs (%.2f GB of cache read per step) exceed the 126 MB L2; no flush needed" % gb,
            "parallelism": "replicas"}


# --------------------------------------------------------------------------------------------
# Replicas: the path has no exchange step, so N GPUs run N independent copies of the batch
# --------------------------------------------------------------------------------------------
class Replicas:
    """One process per GPU.  The only communication is the timing protocol: a barrier on both sides
    of the timed region and the maximum of the measured time over the ranks."""

    def __init__(self, backend="nccl", device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            self.dist = dist
            kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
            dist.init_process_group(backend, **kw)

    def seed_for(self, base_seed):
        """Every replica draws its own batch."""
        return base_seed + 7919 * self.rank

    def barrier(self):
        if self.dist:
            self.dist.barrier()

    def max_over_ranks(self, ms):
        if not self.dist:
            return ms
        import torch
        t = torch.tensor([ms], dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def job_value(self, units_per_rank, ms_step):
        """Whole-job throughput: what all ranks processed divided by the slowest rank's time."""
        return self.world * units_per_rank / (ms_step * 1e-3)

    def close(self):
        if self.dist:
            self.dist.destroy_process_group()


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
def parse_window(args):
    if not args.window or args.mode == "full":
        return None
    window = tuple(int(v) for v in args.window.split(","))
    return window if sum(window) else None


class Run:
    """One workload on one GPU with the options of the command line applied, and the steps that are timed."""

    def __init__(self, w, args, local_rank):
        import torch
        self.torch = torch
        self.w, self.args = w, args
        self.full = args.mode == "full"
        resident, self.step_layers = plan_layers(w, args.mode)
        self.window = parse_window(args)
        self.st = st = State(w, local_rank, resident, self.window)
        self.ctx = ctx = st.ctx
        if args.stored_path is not None:
            ctx.set_stored_path(args.stored_path)
        if args.decode_path is not None and not self.full:
            ctx.set_decode_path(args.decode_path)
        self.absorbed = args.decode_mode == "absorbed" and not self.full
        if self.absorbed:
            ctx.enable_absorbed()
        st.rope = args.rope
        if args.rope:
            ctx.set_rope(args.rope)
        self.n_attend = sum(1 for _, a in self.step_layers if a)
        self.last = [l for l, a in self.step_layers if a][-1]
        # the uncompressed step at the same shape: every layer attends a full cache.  The layers that hold one
        # here are the anchors; a 32-layer step walks them n_layers / n_anchors times.
        anchors = [l for l in resident if w.is_anchor(l)]
        n_layers_step = w.n_layers if w.n_layers > 2 else 1
        self.full_layers = [anchors[i % len(anchors)] for i in range(n_layers_step)]

    def attend(self, l):
        st, ctx = self.st, self.ctx
        if self.full or self.w.is_anchor(l):   # the uncompressed mode / an anchor layer: Eq. 7 on the stored full cache
            ctx.full_attention(l, st.q_dev[l], st.lens, out=st.out[l])
        else:
            ctx.decode_attention(l, st.q_dev[l], st.lens, out=st.out[l])

    def step(self):
        st, ctx = self.st, self.ctx
        for l, a in self.step_layers:
            ctx.append_kv(l, st.new_dev[(l, "k")], st.new_dev[(l, "v")], st.positions)
            if a:
                self.attend(l)

    def step_host(self):
        st, ctx = self.st, self.ctx
        for l, a in self.step_layers:
            ctx.layer_step_host(l, st.q_host[l] if a else None, st.new_host[(l, "k")], st.new_host[(l, "v")],
                                st.out_host[l] if a else None, st.lens_host, attend=a)

    def step_uncompressed(self):
        st, ctx = self.st, self.ctx
        for l in self.full_layers:
            ctx.append_kv(l, st.new_dev[(l, "k")], st.new_dev[(l, "v")], st.positions)
            ctx.full_attention(l, st.q_dev[l], st.lens, out=self.full_out)

    def close(self):
        self.ctx.close()


def timed(run, rep, fn, steps, kernel_timing=True):
    """`steps` calls of fn between two events on torch's current stream (the one every launch goes to), a
    barrier + synchronize on both sides, max over ranks.  Returns (ms total, per-kind kernel times, launches)."""
    torch = run.torch
    ctx = run.ctx

    def sync_all():
        torch.cuda.synchronize()
        if rep.dist:
            rep.barrier()
            torch.cuda.synchronize()

    if kernel_timing:
        ctx.set_kernel_timing(True)
        ctx.read_kernel_timing()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for _ in range(steps):
        fn()
    e1.record()
    sync_all()
    ms_total = rep.max_over_ranks(e0.elapsed_time(e1))
    launches = ctx.launch_count() - launches0
    timing = ctx.read_kernel_timing_by_kind() if kernel_timing else None
    ctx.set_kernel_timing(False)
    return ms_total, timing, launches


def roofline_of(run, args, timing, ms_region, peaks, peaks_kind):
    """The roofline record of the dominant kernel from the per-kind kernel times of a timed region."""
    w, ctx = run.w, run.ctx
    elem = 2 if w.dtype == "bf16" else 4
    flops, bytes_ = algorithmic_work(w)
    stored_ms, stored_n = timing["stored"]
    recon_ms, recon_n = timing["recon"]
    burst_tf = float(peaks["bf16_tflops"])
    sustained_tf = float(peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"])
    tensor_source = ("%s cuBLAS bf16 GEMM, burst figure: the ceiling (a GEMM loop under the power cap -- the "
                     "sustained figure, %.0f TFLOP/s -- is below what this kernel reaches, so it is listed as "
                     "frac_of_sustained_peak only)" % (peaks_kind, sustained_tf))
    full_bytes = w.batch * w.context * 2.0 * w.D * elem   # a stored layer: every K and V row once
    stored_info = None
    if stored_n:
        k_ms = stored_ms / stored_n
        stored_info = {"kernel": stored_kernel_name(ctx),
                       "kernel_ms": k_ms, "kernel_launches": stored_n, "achieved_gbs": full_bytes / (k_ms * 1e-3) / 1e9,
                       "frac_of_%s_hbm" % peaks_kind: full_bytes / (k_ms * 1e-3) / 1e9 / float(peaks["hbm_gbs"])}
    if run.absorbed:
        # the absorbed mode streams [anchor dims ; retained dims] of K once and of V once: HBM-bound; its two
        # streaming kernels are reported together (each moves half of the bytes)
        ak_ms, ak_n = timing["absorb_k"]
        av_ms, av_n = timing["absorb_v"]
        k_ms = (ak_ms + av_ms) / max(ak_n, 1)
        if w.save_k:      # the K pass streams the layer's own D key dims instead of [anchor ; retained]
            bytes_ = w.batch * w.context * float(w.D + w.d_in) * elem
        achieved_gbs = bytes_ / (k_ms * 1e-3) / 1e9
        peak_gbs = float(peaks["hbm_gbs"])
        roofline = {"bound": "hbm", "achieved": achieved_gbs, "peak": peak_gbs, "unit": "GB/s",
                    "frac": achieved_gbs / peak_gbs,
                    "traffic": traffic_of(args, (args.workload or HEADLINE) + "_absorbed"),
                    "kernel": "absorb_scores_kernel + absorb_pv_kernel", "kernel_ms": k_ms,
                    "kernel_ms_k_pass": ak_ms / max(ak_n, 1), "kernel_ms_v_pass": av_ms / max(av_n, 1),
                    "kernel_launches": ak_n + av_n, "share_of_step": (ak_ms + av_ms) / ms_region,
                    "peak_source": "%s (STREAM-style copy)" % peaks_kind,
                    "algorithmic_bytes_per_launch": bytes_,
                    "mode": "absorbed predictors: the same outputs as the explicit path, a separate roofline row"}
        if args.rope and w.save_k:
            roofline["kernel"] = "key_scores_rope_kernel + absorb_pv_kernel"
            roofline["mode"] = "keys kept whole and rotated when read: stored-key scores, V side with absorbed predictors"
        elif args.rope:
            # rotated keys: the K side is explicit (Eq. 3 for the keys on the tensor cores, rotation, scores), only
            # the V side is absorbed; the K pass is the dominant kernel and tensor-bound
            tokens = float(w.batch) * w.context
            k_flops = tokens * 2.0 * w.d_in * w.d_drop
            k_pass_ms = ak_ms / max(ak_n, 1)
            achieved_tf = k_flops / (k_pass_ms * 1e-3) / 1e12
            roofline = {"bound": "tensor", "achieved": achieved_tf, "peak": burst_tf, "unit": "TFLOP/s",
                        "frac": achieved_tf / burst_tf, "frac_of_sustained_peak": achieved_tf / sustained_tf,
                        "traffic": None,
                        "kernel": "recon_pair_kernel (key scores) + key_scores_rope_kernel", "kernel_ms": k_pass_ms,
                        "kernel_ms_k_pass": k_pass_ms, "kernel_ms_v_pass": av_ms / max(av_n, 1),
                        "kernel_launches": ak_n, "share_of_step": ak_ms / ms_region,
                        "peak_source": tensor_source,
                        "algorithmic_flops_per_launch": k_flops,
                        "v_pass_frac_of_hbm": (bytes_ / 2) / (av_ms / max(av_n, 1) * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
                        "mode": "rotated keys: K side explicit, V side with absorbed predictors"}
        if stored_info:
            roofline["anchor_layers"] = stored_info
    elif recon_n:
        k_ms = recon_ms / recon_n
        achieved_tf = flops / (k_ms * 1e-3) / 1e12
        fused_name = fused_kernel_name(ctx)
        fused_traffic = traffic_of(args, args.workload or HEADLINE)
        if (args.workload or HEADLINE) in ("c1", "c3") and not fused_name.startswith("recon_quad"):
            fused_traffic = None          # (the stored figure is a capture of recon_quad_kernel)
        roofline = {"bound": "tensor", "achieved": achieved_tf, "peak": burst_tf, "unit": "TFLOP/s",
                    "frac": achieved_tf / burst_tf, "frac_of_burst_peak": achieved_tf / burst_tf,
                    "frac_of_sustained_peak": achieved_tf / sustained_tf, "peak_sustained": sustained_tf,
                    "traffic": fused_traffic,
                    "kernel": fused_name,
                    "kernel_ms": k_ms, "kernel_launches": recon_n,
                    "share_of_step": recon_ms / ms_region,
                    "peak_source": tensor_source,
                    "algorithmic_flops_per_launch": flops, "algorithmic_bytes_per_launch": bytes_,
                    "hbm_frac_of_%s" % peaks_kind: bytes_ / (k_ms * 1e-3) / 1e9 / float(peaks["hbm_gbs"])}
        if stored_info:
            roofline["anchor_layers"] = stored_info
    else:
        k_ms = stored_ms / max(stored_n, 1)
        achieved_gbs = full_bytes / (k_ms * 1e-3) / 1e9
        peak_gbs = float(peaks["hbm_gbs"])
        roofline = {"bound": "hbm", "achieved": achieved_gbs, "peak": peak_gbs, "unit": "GB/s",
                    "frac": achieved_gbs / peak_gbs, "traffic": traffic_of(args, (args.workload or HEADLINE) + "_full"),
                    "kernel": stored_info["kernel"] if stored_info else None,
                    "kernel_ms": k_ms, "kernel_launches": stored_n, "share_of_step": stored_ms / ms_region,
                    "peak_source": "%s (STREAM-style copy)" % peaks_kind,
                    "algorithmic_bytes_per_launch": full_bytes}
    return roofline


def measure(run, rep, args, steps, warmup, peaks, peaks_kind, with_e2e=True):
    """Warm-up, the device-resident timed region, and the end-to-end region of one workload."""
    torch = run.torch
    w, ctx, st = run.w, run.ctx, run.st
    from paper_2603_22910_b200 import binding
    for _ in range(warmup):
        run.step()
    torch.cuda.synchronize()
    assert ctx.device_status() == binding.ECHOKV_OK, "device status after warm-up"
    sampler = ClockSampler(physical_gpu_index(rep.local_rank))
    sampler.start()
    ms_total, timing, launches = timed(run, rep, run.step, steps)
    ms_eager = ms_total
    if args.graph:
        # the same step captured once in a CUDA graph and replayed: what the launch gaps cost; the per-kernel
        # times above come from the eager pass (events cannot be read out of a captured region)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            run.step()                                   # (first-use set-up of every kernel stays outside the capture)
            side.synchronize()
            with torch.cuda.graph(graph, stream=side):
                run.step()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            graph.replay()
        ms_total, _, _ = timed(run, rep, graph.replay, steps, kernel_timing=False)
    clocks = sampler.stop()
    status = ctx.device_status()
    assert status == binding.ECHOKV_OK, "device status %d after the timed region" % status
    ms_step = ms_total / steps
    rec = {
        "ms_per_step": ms_step,
        "value": rep.job_value(w.batch, ms_step),
        "us_per_layer_step": ms_step * 1e3 / run.n_attend,
        "kv_tokens_scanned_per_s": rep.world * w.batch * w.context * run.n_attend / (ms_step * 1e-3),
        "clocks": clocks,
        "gpu_launches": int(launches),
        "roofline": roofline_of(run, args, timing, ms_eager, peaks, peaks_kind),
        "cuda_graph": {"ms_per_step_eager": ms_eager / steps} if args.graph else None,
    }
    if with_e2e:
        # ---- end to end from pinned host memory ----
        for _ in range(min(3, warmup)):
            run.step_host()
        ms_e2e, _, _ = timed(run, rep, run.step_host, steps, kernel_timing=False)
        elem = 2 if w.dtype == "bf16" else 4
        h2d = (len(run.step_layers) * (2 * w.batch * w.D * elem + 2 * w.batch * 4)
               + run.n_attend * w.batch * w.n_q_heads * w.head_dim * elem)
        d2h = run.n_attend * w.batch * w.n_q_heads * w.head_dim * 4
        same = bool(torch.equal(st.out_host[run.last], st.out[run.last].cpu()))
        rec["e2e"] = {"value": rep.job_value(w.batch, ms_e2e / steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
                      "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e / steps, "matches_device_path": same}
    return rec


def measure_uncompressed(run, rep, steps, peaks, peaks_kind):
    """The uncompressed step at the same shape (every layer attends a full cache), beside the compressed one."""
    torch = run.torch
    w = run.w
    if run.full:
        return None
    run.full_out = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32, device=run.st.dev)
    for _ in range(3):
        run.step_uncompressed()
    ms_total, timing, _ = timed(run, rep, run.step_uncompressed, steps)
    stored_ms, stored_n = timing["stored"]
    elem = 2 if w.dtype == "bf16" else 4
    full_bytes = w.batch * w.context * 2.0 * w.D * elem
    k_ms = stored_ms / max(stored_n, 1)
    gbs = full_bytes / (k_ms * 1e-3) / 1e9
    return {"ms_per_step": ms_total / steps, "layers_per_step": len(run.full_layers),
            "kernel": stored_kernel_name(run.ctx),
            "kernel_ms": k_ms, "achieved_gbs": gbs, "frac_of_%s_hbm" % peaks_kind: gbs / float(peaks["hbm_gbs"]),
            "what": "full-cache attention on every layer of the step (the layers that hold a full cache here, "
                    "walked %d time(s))" % (len(run.full_layers) // max(1, len(set(run.full_layers))))}


def fused_kernel_name(ctx):
    """The fused reconstruct-then-attend kernel that served the last decode call of this context."""
    path = ctx.decode_path()
    if path == 5:      # chosen on the device by the page order of the block table
        return "recon_tc_kernel (pages in order)" if ctx.diag_page_order() == 1 else "recon_quad_kernel (pages out of order)"
    return {4: "recon_quad_kernel", 3: "recon_pair_kernel", 2: "recon_tc_kernel"}.get(path, "recon_simt_kernel")


def stored_kernel_name(ctx):
    """The kernel that serves stored heads in this context (csrc/stored_mma.cu, csrc/simt_kernels.cu)."""
    if ctx.stored_path() != 1:
        return "attn_stored_kernel"
    return "attn_stored_rope_kernel" if ctx.rope_enabled() else "attn_stored_mma_kernel"


def sustained_leg(run, rep, ms_step, seconds, peaks, peaks_kind, args):
    """The step repeated for at least `seconds`, with its own kernel times and clock samples."""
    steps = max(3, int(math.ceil(seconds * 1e3 / ms_step)))
    sampler = ClockSampler(physical_gpu_index(rep.local_rank))
    sampler.start()
    ms_total, timing, _ = timed(run, rep, run.step, steps)
    clocks = sampler.stop()
    roof = roofline_of(run, args, timing, ms_total, peaks, peaks_kind)
    out = {"seconds": ms_total * 1e-3, "steps": steps, "ms_per_step": ms_total / steps,
           "value": rep.job_value(run.w.batch, ms_total / steps), "kernel": roof.get("kernel"),
           "kernel_ms": roof.get("kernel_ms"), "frac": roof.get("frac"), "unit": roof.get("unit"),
           "achieved": roof.get("achieved"), "clocks": clocks}
    for k in ("frac_of_burst_peak", "frac_of_sustained_peak", "anchor_layers"):
        if k in roof:
            out[k] = roof[k]
    if clocks.get("sm_mhz") and roof.get("kernel_ms"):
        # time x clock: compares kernels measured at different clocks (NVML's reading of the SM clock)
        out["kernel_ms_x_sm_mhz"] = roof["kernel_ms"] * clocks["sm_mhz"]
    return out


def sub_args(args, **kw):
    a = argparse.Namespace(**vars(args))
    a.batch = a.context = a.page_tokens = 0
    a.random_pages = False
    a.ratio = 75
    for k, v in kw.items():
        setattr(a, k, v)
    return a


def run_suite(args, rep, peaks, peaks_kind):
    """The default run: headline + sustained leg + one sub-record per benchmark configuration."""
    import torch
    from paper_2603_22910_b200 import binding
    line, configs = None, {}
    order = [HEADLINE] + [k for k, _ in SUITE if k != HEADLINE]
    specs = dict(SUITE)
    single_gpu = rep.world == 1
    for key in order:
        if key != HEADLINE and not single_gpu:
            break                                  # the sub-records are a one-GPU matter
        a = sub_args(args, **specs[key])
        w = workload_of_args(a)
        w = w.replace(seed=rep.seed_for(w.seed))
        run = Run(w, a, rep.local_rank)
        steps = args.steps if key == HEADLINE else max(10, min(args.steps, 30))
        if w.n_layers > 2 and key != HEADLINE:
            steps = min(steps, 10)
        rec = measure(run, rep, a, steps, args.warmup, peaks, peaks_kind)
        rec["steps"] = steps
        rec["config"] = workload_config(w)
        rec["decode_path"] = run.ctx.decode_path()
        if key == HEADLINE or key == "c2":
            # (the GQA backbone shape too: its short timed region ends before the power cap has settled)
            rec["sustained"] = sustained_leg(run, rep, rec["ms_per_step"], args.sustained_s, peaks, peaks_kind, a)
        if single_gpu and rep.rank == 0:
            run.step()
            torch.cuda.synchronize()
            picks = stratified_picks(w, [l for l, at in run.step_layers if at], 8, seed=11, max_combos=2)
            rec["parity_vs_oracle"] = parity_sample(run.st, picks)
            if key == HEADLINE and not args.no_cpu_baseline:
                cpu_value, sample, _ = time_oracle(run.st, run.step_layers, budget_s=10.0)
                rec["cpu_baseline"] = {"value": cpu_value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                       "sample": sample}
            rec["uncompressed"] = measure_uncompressed(run, rep, steps, peaks, peaks_kind)
        assert run.ctx.device_status() == binding.ECHOKV_OK
        rec["input_generation_s"] = run.st.gen_s
        configs[key] = rec
        if key == HEADLINE:
            line = headline_line(rec, w, a, rep, args, run)
        run.close()
        del run
        torch.cuda.empty_cache()
    if single_gpu:
        line["configs"] = {k: summary_of(v) for k, v in configs.items()}
    return line


def summary_of(rec):
    r = rec["roofline"]
    out = {"workload": rec["config"]["workload"], "steps": rec["steps"], "ms_per_step": rec["ms_per_step"],
           "tokens_per_s": rec["value"], "e2e_ms_per_step": rec["e2e"]["ms_per_step"],
           "e2e_tokens_per_s": rec["e2e"]["value"], "kernel": r.get("kernel"), "kernel_ms": r.get("kernel_ms"),
           "bound": r.get("bound"), "achieved": r.get("achieved"), "unit": r.get("unit"),
           "frac_of_burst_peak": r.get("frac_of_burst_peak"), "frac_of_sustained_peak": r.get("frac_of_sustained_peak"),
           "algorithmic_flops_per_launch": r.get("algorithmic_flops_per_launch"),
           "clocks": rec["clocks"], "parity_vs_oracle": rec.get("parity_vs_oracle"),
           "uncompressed": rec.get("uncompressed")}
    if "anchor_layers" in r:
        out["anchor_layers"] = r["anchor_layers"]
    if "sustained" in rec:
        out["sustained"] = rec["sustained"]
    return out


def headline_line(rec, w, a, rep, args, run):
    line = {
        "metric": METRIC, "value": rec["value"], "unit": UNIT, "n_gpus": rep.world, "steps": rec.get("steps", args.steps),
        "warmup": args.warmup, "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": workload_config(w, run.full),
        "us_per_layer_step": rec["us_per_layer_step"],
        "kv_tokens_scanned_per_s": rec["kv_tokens_scanned_per_s"],
        "clocks": rec["clocks"],
        "e2e": rec["e2e"],
        "gpu_launches": rec["gpu_launches"],
        "roofline": rec["roofline"],
        "decode_path": run.ctx.decode_path(), "stored_path": run.ctx.stored_path(),
        "decode_mode": "absorbed" if run.absorbed else "explicit",
        "cuda_graph": rec["cuda_graph"],
        "full_precision_tokens": {"sink": run.window[0], "window": run.window[1]} if run.window else None,
        "rope_theta": a.rope or None,
        "input_generation_s": run.st.gen_s,
    }
    for k in ("sustained", "cpu_baseline", "parity_vs_oracle"):
        if k in rec:
            line[k] = rec[k]
    return line


def run_single(args, rep, peaks, peaks_kind):
    """--workload given: that workload alone, with the command line's options."""
    import numpy as np
    import torch
    w = workload_of_args(args)
    w = w.replace(seed=rep.seed_for(w.seed))
    run = Run(w, args, rep.local_rank)
    rec = measure(run, rep, args, args.steps, args.warmup, peaks, peaks_kind)
    rec["steps"] = args.steps
    if args.sustained_s > 0:
        rec["sustained"] = sustained_leg(run, rep, rec["ms_per_step"], args.sustained_s, peaks, peaks_kind, args)
    if rep.rank == 0 and rep.world == 1 and not args.no_cpu_baseline:
        st = run.st
        cpu_value, sample, outs = time_oracle(st, run.step_layers, budget_s=12.0)
        worst_abs, num, den = 0.0, 0.0, 0.0
        for (l, b), ref in outs.items():
            gpu = st.out[l][b].cpu().numpy().astype(np.float64)
            worst_abs = max(worst_abs, float(np.max(np.abs(gpu - ref))))
            num += float(np.sum((gpu - ref) ** 2))
            den += float(np.sum(ref ** 2))
        rec["cpu_baseline"] = {"value": cpu_value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                               "sample": sample}
        rec["parity_vs_oracle"] = {"outputs": sorted(outs.keys()), "max_abs": worst_abs,
                                   "rel_l2": (num / max(den, 1e-300)) ** 0.5}
    line = headline_line(rec, w, args, rep, args, run)
    run.close()
    return line


def graph_replay_ms(run, rep, steps):
    """The step captured once in a CUDA graph and replayed: what a serving loop that captures its decode step pays
    (the launch gaps between the kernels of a short step are what it removes)."""
    torch = run.torch
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        run.step()                                   # (first-use set-up of every kernel stays outside the capture)
        side.synchronize()
        with torch.cuda.graph(graph, stream=side):
            run.step()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(3):
        graph.replay()
    ms_total, _, _ = timed(run, rep, graph.replay, steps, kernel_timing=False)
    del graph
    return ms_total / steps


def run_sweep(args, rep, peaks, peaks_kind):
    """--workload c4 --sweep: every point of the sweep that fits the device, explicit, absorbed and uncompressed
    steps side by side, each against its own roofline."""
    import torch
    points = []
    burst = float(peaks["bf16_tflops"])
    sustained = float(peaks.get("bf16_tflops_sustained") or burst)
    hbm = float(peaks["hbm_gbs"])
    ratios = [int(v) for v in args.sweep_ratios.split(",")]
    contexts = [int(v) for v in args.sweep_contexts.split(",")]
    batches = [int(v) for v in args.sweep_batches.split(",")]
    for ratio in ratios:
        for L in contexts:
            for B in batches:
                a = sub_args(args, workload="c4", ratio=ratio, context=L, batch=B)
                w = workload_of_args(a)
                cache_gb = B * L * 2 * (w.D + w.d_in) * 2 / 1e9      # anchor + compressed layer pools
                if cache_gb > 120:
                    points.append({"ratio": ratio, "context": L, "batch": B, "skipped": "%.0f GB of cache" % cache_gb})
                    continue
                run = Run(w, a, rep.local_rank)
                steps = 20 if B * L <= 2 ** 20 else 8
                for _ in range(3):
                    run.step()
                ms_exp, timing, _ = timed(run, rep, run.step, steps)
                small = B * L <= 2 ** 17         # short steps: also replayed from a CUDA graph
                ms_exp_graph = graph_replay_ms(run, rep, steps) if small else None
                ref = run.st.out[1].clone()
                run.full_out = torch.empty_like(ref)
                for _ in range(3):
                    run.step_uncompressed()
                ms_full, timing_full, _ = timed(run, rep, run.step_uncompressed, steps)
                run.ctx.enable_absorbed()
                for _ in range(3):
                    run.step()
                ms_abs, _, _ = timed(run, rep, run.step, steps)
                diff = float((run.st.out[1] - ref).norm() / ref.norm())
                ms_abs_graph = graph_replay_ms(run, rep, steps) if small else None
                status = run.ctx.device_status()
                flops, bytes_ = algorithmic_work(w)
                recon_ms, recon_n = timing["recon"]
                k_ms = recon_ms / max(recon_n, 1)
                full_bytes = B * L * 2.0 * w.D * 2
                points.append({
                    "ratio": ratio, "context": L, "batch": B, "decode_path": run.ctx.decode_path(),
                    "ms_explicit": ms_exp / steps, "kernel_ms": k_ms,
                    "kernel_frac_of_burst_peak": flops / (k_ms * 1e-3) / 1e12 / burst,
                    "step_frac_of_burst_peak": flops / (ms_exp / steps * 1e-3) / 1e12 / burst,
                    "step_frac_of_sustained_peak": flops / (ms_exp / steps * 1e-3) / 1e12 / sustained,
                    "ms_absorbed": ms_abs / steps, "absorbed_step_frac_of_hbm": bytes_ / (ms_abs / steps * 1e-3) / 1e9 / hbm,
                    "ms_uncompressed": ms_full / steps,
                    "uncompressed_step_frac_of_hbm": full_bytes / (ms_full / steps * 1e-3) / 1e9 / hbm,
                    "rel_l2_absorbed_vs_explicit": diff, "device_status": status})
                if small:
                    points[-1].update({
                        "ms_explicit_graph": ms_exp_graph,
                        "step_frac_of_burst_peak_graph": flops / (ms_exp_graph * 1e-3) / 1e12 / burst,
                        "ms_absorbed_graph": ms_abs_graph,
                        "absorbed_step_frac_of_hbm_graph": bytes_ / (ms_abs_graph * 1e-3) / 1e9 / hbm})
                run.close()
                del run, ref
                torch.cuda.empty_cache()
    done = [p for p in points if "ms_explicit" in p]
    last = done[-1]
    return {"metric": METRIC, "value": last["batch"] / (last["ms_explicit"] * 1e-3), "unit": UNIT, "n_gpus": rep.world,
            "steps": 20, "warmup": 3, "ms_per_step": last["ms_explicit"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "c4 sweep on the Llama-3-8B layer shape: ratios %s x contexts %s x batches %s; "
                                   "value / ms_per_step are the last point's" % (ratios, contexts, batches),
                       "parallelism": "one GPU"},
            "peaks": {"bf16_tflops_burst": burst, "bf16_tflops_sustained": sustained, "hbm_gbs": hbm,
                      "source": peaks_kind},
            "sweep": points}


def run_ours(args):
    import torch
    from paper_2603_22910_b200 import binding, build

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    rep = Replicas("nccl", torch.device("cuda", local_rank))
    if rep.rank == 0:
        build.build()
    rep.barrier()
    binding.lib()
    peaks, peaks_kind = load_peaks()
    if args.sweep:
        line = run_sweep(args, rep, peaks, peaks_kind)
    elif args.workload is None:
        line = run_suite(args, rep, peaks, peaks_kind)
    else:
        line = run_single(args, rep, peaks, peaks_kind)
    if rep.rank == 0:
        print(json.dumps(line))
    rep.close()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=None, choices=["c1", "c2", "c3", "c4"],
                    help="default: the whole record (headline c3, the 32-layer decode step, plus one sub-record per "
                         "configuration).  c1: Llama-2-7B-shaped layer; c2: Llama-3-8B-shaped GQA layer; c3: 32-layer "
                         "Llama-2-7B-shaped decode step; c4: one point of the GQA sweep (--ratio, --context, --batch)")
    ap.add_argument("--mode", default="compressed", choices=["compressed", "full"],
                    help="compressed: decode attention of a compressed layer (the headline); full: the "
                         "uncompressed path, full-cache attention on the anchor layer")
    ap.add_argument("--sweep", action="store_true", help="with --workload c4: the whole sweep, one sub-record per point")
    ap.add_argument("--sweep-ratios", default="25,50,75")
    ap.add_argument("--sweep-contexts", default="4096,16384,65536,131072")
    ap.add_argument("--sweep-batches", default="1,8,32,64")
    ap.add_argument("--sustained-s", type=float, default=None,
                    help="repeat the step for at least this many seconds after the timed steps, with the clocks "
                         "sampled (default 2 for the whole record, 0 with --workload)")
    ap.add_argument("--stored-path", type=int, default=None, choices=[0, 1],
                    help="kernel for stored heads: 0 CUDA-core, 1 TMA + tensor-core (default: the library's choice)")
    ap.add_argument("--decode-path", type=int, default=None, choices=[1, 2, 3, 4, 5],
                    help="kernel family for compressed layers (default: the library's choice)")
    ap.add_argument("--decode-mode", default="explicit", choices=["explicit", "absorbed"],
                    help="explicit: reconstruct-then-attend as the paper states it (the headline); absorbed: the "
                         "predictors folded into the queries and the output (same outputs, HBM-bound)")
    ap.add_argument("--graph", action="store_true",
                    help="time the step replayed from a CUDA graph (launch gaps removed) instead of eager launches")
    ap.add_argument("--window", default="", help="n_sink,n_window: tokens kept at full precision, e.g. 4,128 (the "
                                                 "paper's setting); default none, as the benchmark configs state")
    ap.add_argument("--rope", type=float, default=0.0, help="theta of a rotary embedding applied when the cache is "
                    "read (the cache then holds un-rotated keys); 0 = none, as in the paper's configurations")
    ap.add_argument("--save-k", action="store_true", help="compressed layers keep their keys whole, only the values "
                    "are predicted (the paper's \"save K\" ablation)")
    ap.add_argument("--prefill-queries", type=int, default=0, help="time the prefill-shaped call instead: this many "
                    "causal queries per sequence on the compressed layer (an extra measurement, its own JSON line)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling a smaller case)")
    ap.add_argument("--context", type=int, default=0, help="override the workload's context length")
    ap.add_argument("--ratio", type=int, default=75, choices=[25, 50, 75],
                    help="c4 only: percent of the layer's KV heads discarded")
    ap.add_argument("--retained-dims", type=int, default=0,
                    help="c4 only: m in flat dims instead of --ratio, e.g. 64 or 384 (the paper's settings)")
    ap.add_argument("--page-tokens", type=int, default=0, choices=[0, 16, 32, 64, 128],
                    help="override the tokens per cache page (default 16)")
    ap.add_argument("--random-pages", action="store_true", help="pages of the pool in a seeded random order")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.sustained_s is None:
        args.sustained_s = 2.0 if args.workload is None else 0.0
    if args.impl == "reference":
        return run_reference(args)
    if args.prefill_queries:
        if args.workload is None:
            args.workload = "c2"
        return run_prefill(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
