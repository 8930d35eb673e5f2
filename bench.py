#!/usr/bin/env python
"""Benchmark of the EchoKV decode path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c2] [--impl ours|reference]

One "step" = one pass of the whole hot path over one batch of synthetic input:
append the new token to the anchor layer and to the compressed layer (which keeps
only the retained heads), then decode attention on the compressed layer -- retained
heads from the cache, dropped heads reconstructed on chip -- including the split-K
merge.  `value` is decode tokens per second (sequences advanced per second) with the
caches resident in HBM; `e2e` is the same step driven from pinned host buffers
through echokv_layer_step_host.  With N > 1 every rank runs an independent replica
of the batch (the path has no exchange step): weak scaling, no collective on the
data path.

--impl reference times the CPU oracle (numpy, fp64) on a bounded sample of the same
workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"

# DRAM bytes per launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum) from
# the ncu captures summarised under profiles/; None until a capture of that workload exists.
NCU_TRAFFIC_BYTES = {"c1": None, "c2": None}

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def workload_by_name(name, batch=0, context=0):
    from paper_2603_22910_b200 import synth
    w = {"c1": synth.C1, "c2": synth.C2, "c0": synth.C0}[name]
    if batch:
        w = w.replace(batch=batch, name=w.name + "_B%d" % batch)
    if context:
        w = w.replace(context=context, name=w.name + "_L%d" % context)
    return w


def algorithmic_work(w):
    """Per launch of the fused kernel: FLOPs of Eq. 3 (both predictors) plus Eq. 7 on the dropped
    heads, and the bytes the method must move (predictor inputs once, predictors once)."""
    tokens = w.batch * w.context
    g = w.n_q_heads // w.n_kv_heads
    n_drop_q = (w.n_kv_heads - w.n_retained_heads) * g
    flops = tokens * (4.0 * w.d_in * w.d_drop + 4.0 * n_drop_q * w.head_dim)
    elem = 2 if w.dtype == "bf16" else 4
    bytes_ = tokens * 2.0 * w.d_in * elem + 2.0 * w.d_in * w.d_drop * elem
    return flops, bytes_


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index = index
        self.samples, self.reasons = [], set()
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
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                for bit, name in names.items():
                    if mask & bit and name != "gpu_idle":
                        self.reasons.add(name)
                time.sleep(0.004)
        except Exception as e:  # NVML missing: report it rather than guess
            self.error = repr(e)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2.0)
        s = sorted(self.samples)
        med = s[len(s) // 2] if s else None
        out = {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(s)}
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


def oracle_inputs(w, layer, b):
    """Widened (float64) oracle inputs of sequence b from the seeded generators."""
    from oracle import echokv_oracle as O
    from paper_2603_22910_b200 import synth
    a = w.anchor_of(layer)
    st = synth.to_numpy_stored
    kg = O.widen(st(synth.layer_cache(w, a, "k", b)))
    vg = O.widen(st(synth.layer_cache(w, a, "v", b)))
    kl = O.widen(st(synth.layer_cache(w, layer, "k", b, width=w.m)))
    vl = O.widen(st(synth.layer_cache(w, layer, "v", b, width=w.m)))
    Wk = O.widen(st(synth.predictor_weights(w, layer, "k")))
    Wv = O.widen(st(synth.predictor_weights(w, layer, "v")))
    q = O.widen(st(synth.queries(w, layer)))[b]
    return q, kg, vg, kl, vl, Wk, Wv


def time_oracle(w, budget_s, max_seqs=None, full=False):
    """The oracle as it stands on whole sequences of the workload until `budget_s` is used."""
    from oracle import echokv_oracle as O
    layer = 1
    done, elapsed = 0, 0.0
    outs = {}
    for b in range(w.batch if max_seqs is None else min(w.batch, max_seqs)):
        args = oracle_inputs(w, layer, b)
        t0 = time.perf_counter()
        if full:     # the anchor layer's stored cache
            outs[b] = O.full_attention(args[0], args[1], args[2], w.n_kv_heads)
        else:
            outs[b] = O.decode_attention(*args, n_kv_heads=w.n_kv_heads)
        elapsed += time.perf_counter() - t0
        done += 1
        if elapsed >= budget_s:
            break
    return done, elapsed, outs


def run_reference(args):
    """--impl reference: the CPU oracle, as it stands, on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    from oracle import echokv_oracle as O
    w = workload_by_name(args.workload, args.batch, args.context)
    layer = 1
    g = w.n_q_heads // w.n_kv_heads
    dropped_q = list(range(w.n_retained_heads * g, w.n_q_heads))
    inputs = oracle_inputs(w, layer, 0)
    # probe: one dropped KV head's query heads on sequence 0
    probe_heads = dropped_q[:g]
    t0 = time.perf_counter()
    O.decode_attention_query_heads(*inputs, n_kv_heads=w.n_kv_heads, query_heads=probe_heads)
    t_head = time.perf_counter() - t0
    total = args.steps + args.warmup
    budget = 150.0
    n_kv_sample = max(1, min(w.n_kv_heads - w.n_retained_heads, int(budget / max(total * t_head, 1e-9))))
    heads = dropped_q[: n_kv_sample * g]
    times = []
    for i in range(total):
        t0 = time.perf_counter()
        O.decode_attention_query_heads(*inputs, n_kv_heads=w.n_kv_heads, query_heads=heads)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    # a step covers n_kv_sample of the (H_kv - r) dropped heads of ONE of the B sequences; the
    # retained heads cost next to nothing beside them, so a whole batch step takes about
    # B * (H_kv - r) / n_kv_sample times as long
    frac = n_kv_sample / float(w.n_kv_heads - w.n_retained_heads)
    t_step = sum(times) / len(times)
    t_batch = t_step / frac * w.batch
    value = w.batch / t_batch
    sample = ("sequence 0 of %d, %d of %d dropped KV heads per step (all %d tokens), scaled to the full batch"
              % (w.batch, n_kv_sample, w.n_kv_heads - w.n_retained_heads, w.context))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t_batch * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))
    return 0


def workload_config(w, full=False):
    elem = 2 if w.dtype == "bf16" else 4
    if full:
        what = ("%s, uncompressed: B=%d L=%d H_q=%d H_kv=%d d=%d, %s, %d-token pages, full-cache attention on the "
                "anchor layer" % (w.name, w.batch, w.context, w.n_q_heads, w.n_kv_heads, w.head_dim, w.dtype,
                                  w.page_tokens))
        gb = w.batch * w.context * 2 * w.D * elem / 1e9
    else:
        what = ("%s: B=%d L=%d H_q=%d H_kv=%d d=%d retained=%d (D_in=%d -> D_drop=%d), %s, %d-token pages, "
                "anchor + compressed layer" % (w.name, w.batch, w.context, w.n_q_heads, w.n_kv_heads, w.head_dim,
                                               w.n_retained_heads, w.d_in, w.d_drop, w.dtype, w.page_tokens))
        gb = w.batch * w.context * 2 * w.d_in * elem / 1e9
    return {"workload": what, "global_batch": w.batch, "context": w.context,
            "l2": "inputs (%.2f GB of cache per step) exceed the 126 MB L2; no flush needed" % gb,
            "parallelism": "replicas"}


# --------------------------------------------------------------------------------------------
# GPU arm
# --------------------------------------------------------------------------------------------
def run_ours(args):
    import numpy as np
    import torch
    from paper_2603_22910_b200 import binding, build, synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if rank == 0:
        build.build()
    if dist:
        dist.barrier()
    binding.lib()

    w = workload_by_name(args.workload, args.batch, args.context)
    if world > 1:
        w = w.replace(seed=w.seed + 7919 * rank)   # every replica has its own batch
    dev = torch.device("cuda", local_rank)
    cfg = binding.config_for(w, device=local_rank)
    ctx = binding.Context(cfg)
    table = synth.block_table(w)
    ctx.set_block_table(table)
    anchor_l, layer = 0, 1
    # caches: generated per sequence on the host with the seeded generators, laid out in pages
    t_gen = time.perf_counter()
    new = {(l, kind): torch.zeros((w.batch, w.D), dtype=synth.torch_dtype(w)) for l in (anchor_l, layer)
           for kind in ("k", "v")}
    for kind, pools in (("k", ctx.k_pools), ("v", ctx.v_pools)):
        for b in range(w.batch):
            anchor_f32 = synth.anchor_cache(w, anchor_l, kind, b)
            ids = table[b].long().to(dev)
            for l, width in ((anchor_l, w.D), (layer, w.m)):
                if width == 0:
                    continue
                x = synth.layer_cache(w, l, kind, b, width=width, anchor_f32=anchor_f32)
                pools[l][ids] = x.reshape(w.pages_per_seq, w.page_tokens, width).to(dev)
                new[(l, kind)][b, :width] = x[-1]      # the step re-appends the newest token
            del anchor_f32
    new = {k: v.pin_memory() for k, v in new.items()}
    Wk = synth.predictor_weights(w, layer, "k").to(dev)
    Wv = synth.predictor_weights(w, layer, "v").to(dev)
    ctx.set_weights(layer, Wk, Wv)
    q_host = synth.queries(w, layer).pin_memory()
    lens_host = torch.full((w.batch,), w.context, dtype=torch.int32).pin_memory()
    out_host = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32).pin_memory()
    q = q_host.to(dev)
    new_dev = {k: v.to(dev) for k, v in new.items()}
    lens = lens_host.to(dev)
    positions = lens - 1
    out = torch.empty((w.batch, w.n_q_heads, w.head_dim), dtype=torch.float32, device=dev)
    t_gen = time.perf_counter() - t_gen

    full = args.mode == "full"
    if args.stored_path is not None:
        ctx.set_stored_path(args.stored_path)

    def step():
        ctx.append_kv(anchor_l, new_dev[(anchor_l, "k")], new_dev[(anchor_l, "v")], positions)
        if full:     # the uncompressed mode / an anchor layer: Eq. 7 on the stored full cache
            ctx.full_attention(anchor_l, q, lens, out=out)
            return
        ctx.append_kv(layer, new_dev[(layer, "k")], new_dev[(layer, "v")], positions)
        ctx.decode_attention(layer, q, lens, out=out)

    def step_host():
        if full:
            ctx.layer_step_host(anchor_l, q_host, new[(anchor_l, "k")], new[(anchor_l, "v")], out_host, lens_host,
                                attend=True)
            return
        ctx.layer_step_host(anchor_l, None, new[(anchor_l, "k")], new[(anchor_l, "v")], None, lens_host, attend=False)
        ctx.layer_step_host(layer, q_host, new[(layer, "k")], new[(layer, "v")], out_host, lens_host, attend=True)

    def sync_all():
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
            torch.cuda.synchronize()

    def max_over_ranks(ms):
        if not dist:
            return ms
        t = torch.tensor([ms], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    for _ in range(args.warmup):
        step()
    sync_all()
    assert ctx.device_status() == binding.ECHOKV_OK, "device status after warm-up"

    # ---- device-resident timed region -------------------------------------------------------
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    ctx.set_kernel_timing(True)
    ctx.read_kernel_timing()
    launches0 = ctx.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sync_all()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    sync_all()
    ms_total = max_over_ranks(e0.elapsed_time(e1))
    launches = ctx.launch_count() - launches0
    kernel_ms, kernel_launches = ctx.read_kernel_timing()
    ctx.set_kernel_timing(False)
    clocks = sampler.stop()
    status = ctx.device_status()
    assert status == binding.ECHOKV_OK, "device status %d after the timed region" % status

    # ---- end to end from pinned host memory -----------------------------------------------
    for _ in range(min(3, args.warmup)):
        step_host()
    sync_all()
    e2, e3 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e2.record()
    for _ in range(args.steps):
        step_host()
    e3.record()
    sync_all()
    ms_e2e = max_over_ranks(e2.elapsed_time(e3))
    elem = 2 if w.dtype == "bf16" else 4
    n_host_layers = 1 if full else 2
    h2d = (n_host_layers * 2 * w.batch * w.D * elem + w.batch * w.n_q_heads * w.head_dim * elem
           + n_host_layers * 2 * w.batch * 4)
    d2h = w.batch * w.n_q_heads * w.head_dim * 4
    same = bool(torch.equal(out_host, out.cpu()))

    ms_step = ms_total / args.steps
    value = world * w.batch / (ms_step * 1e-3)
    e2e_value = world * w.batch / (ms_e2e / args.steps * 1e-3)

    peaks, peaks_kind = load_peaks()
    flops, bytes_ = algorithmic_work(w)
    k_ms = kernel_ms / max(kernel_launches, 1)
    if full:
        # Eq. 7 on the stored cache: every token's K and V row of every KV head is read once
        bytes_ = w.batch * w.context * 2.0 * w.D * elem
        achieved_gbs = bytes_ / (k_ms * 1e-3) / 1e9
        peak_gbs = float(peaks["hbm_gbs"])
        roofline = {"bound": "hbm", "achieved": achieved_gbs, "peak": peak_gbs, "unit": "GB/s",
                    "frac": achieved_gbs / peak_gbs, "traffic": NCU_TRAFFIC_BYTES.get(args.workload + "_full"),
                    "kernel": "attn_stored_mma_kernel" if ctx.stored_path() == 1 else "attn_stored_kernel",
                    "kernel_ms": k_ms, "kernel_launches": kernel_launches,
                    "peak_source": "%s (STREAM-style copy)" % peaks_kind,
                    "algorithmic_bytes_per_launch": bytes_}
    else:
        achieved_tf = flops / (k_ms * 1e-3) / 1e12
        peak_tf = float(peaks.get("bf16_tflops_sustained") or peaks["bf16_tflops"])
        roofline = {"bound": "tensor", "achieved": achieved_tf, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": achieved_tf / peak_tf, "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
                    "kernel": "recon_tc_kernel", "kernel_ms": k_ms, "kernel_launches": kernel_launches,
                    "peak_source": "%s (bf16 sustained; kernel timed inside a long step)" % peaks_kind,
                    "algorithmic_flops_per_launch": flops, "algorithmic_bytes_per_launch": bytes_,
                    "hbm_frac_of_%s" % peaks_kind: bytes_ / (k_ms * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
                    "frac_of_burst_peak": achieved_tf / float(peaks["bf16_tflops"])}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
        "config": workload_config(w, full),
        "us_per_layer_step": ms_step * 1e3,
        "kv_tokens_scanned_per_s": world * w.batch * w.context / (ms_step * 1e-3),
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": ms_e2e / args.steps, "matches_device_path": same},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "decode_path": ctx.decode_path(), "stored_path": ctx.stored_path(),
        "input_generation_s": t_gen,
    }

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_seq, t_cpu, outs = time_oracle(w, budget_s=12.0, max_seqs=4, full=full)
        gpu = out.cpu().numpy().astype(np.float64)
        worst_abs, num, den = 0.0, 0.0, 0.0
        for b, ref in outs.items():
            worst_abs = max(worst_abs, float(np.max(np.abs(gpu[b] - ref))))
            num += float(np.sum((gpu[b] - ref) ** 2))
            den += float(np.sum(ref ** 2))
        line["cpu_baseline"] = {"value": n_seq / t_cpu, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                "sample": "%d of %d sequences of the batch, all heads, all %d tokens (%.1f s)"
                                          % (n_seq, w.batch, w.context, t_cpu)}
        line["parity_vs_oracle"] = {"sequences": n_seq, "max_abs": worst_abs, "rel_l2": (num / max(den, 1e-300)) ** 0.5}
    if rank == 0:
        print(json.dumps(line))
    ctx.close()
    if dist:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default="c1", choices=["c1", "c2"])
    ap.add_argument("--mode", default="compressed", choices=["compressed", "full"],
                    help="compressed: decode attention of a compressed layer (the headline); full: the "
                         "uncompressed path, full-cache attention on the anchor layer")
    ap.add_argument("--stored-path", type=int, default=None, choices=[0, 1],
                    help="kernel for stored heads: 0 CUDA-core, 1 TMA + tensor-core (default: the library's choice)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling a smaller case)")
    ap.add_argument("--context", type=int, default=0, help="override the workload's context length")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
