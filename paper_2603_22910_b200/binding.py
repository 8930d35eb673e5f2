"""ctypes binding of libechokv.so: the same names as include/echokv.h, argument
marshalling only.  Every step of the decode path runs in the library's CUDA
kernels; PyTorch is used by `Context` for device memory and streams.

The library must have been built (python -m paper_2603_22910_b200.build);
loading fails loudly otherwise -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import math
import os

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libechokv.so")

ECHOKV_BF16, ECHOKV_FP32 = 0, 1
ECHOKV_OK = 0
ECHOKV_EINVAL, ECHOKV_ENOTANCHOR, ECHOKV_ENOTCOMPRESSED, ECHOKV_ECAPACITY = -1, -2, -3, -4
ECHOKV_ENOWEIGHTS, ECHOKV_ECUDA, ECHOKV_ETIMEOUT, ECHOKV_EBADPAGE = -5, -6, -7, -8
ECHOKV_EUNSUPPORTED, ECHOKV_ENOTABLE, ECHOKV_EBADLENGTH, ECHOKV_ESCRATCH = -9, -10, -11, -12


class echokv_config(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("group_size", C.c_int32), ("n_retained_heads", C.c_int32),
                ("page_tokens", C.c_int32), ("max_batch", C.c_int32), ("max_pages_per_seq", C.c_int32),
                ("dtype", C.c_int32), ("n_pages", C.c_int64), ("softmax_scale", C.c_float),
                ("device", C.c_int32), ("n_retained_dims", C.c_int32), ("save_k", C.c_int32)]


class echokv_sizes(C.Structure):
    _fields_ = [("anchor_pool_bytes", C.c_uint64), ("compressed_pool_bytes", C.c_uint64),
                ("block_table_bytes", C.c_uint64), ("workspace_bytes", C.c_uint64),
                ("max_partials", C.c_int32), ("reserved", C.c_int32)]


class echokv_buffers(C.Structure):
    _fields_ = [("k_pools", C.POINTER(C.c_void_p)), ("v_pools", C.POINTER(C.c_void_p)),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_uint64)]


EXPORTS = {
    # name: (restype, argtypes)
    "echokv_query_sizes": (C.c_int, [C.POINTER(echokv_config), C.POINTER(echokv_sizes)]),
    "echokv_create": (C.c_int, [C.POINTER(echokv_config), C.POINTER(echokv_buffers), C.POINTER(C.c_void_p)]),
    "echokv_destroy": (None, [C.c_void_p]),
    "echokv_set_weights": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "echokv_set_block_table": (C.c_int, [C.c_void_p, C.c_void_p]),
    "echokv_append_kv": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_int, C.c_void_p]),
    "echokv_append_kv_chunk": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_int, C.c_int, C.c_void_p]),
    "echokv_compress_layer": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_int, C.c_void_p]),
    "echokv_decode_attention": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_int, C.c_void_p]),
    "echokv_full_attention": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                        C.c_void_p, C.c_int, C.c_void_p]),
    "echokv_prefill_scratch_bytes": (C.c_int, [C.POINTER(echokv_config), C.POINTER(C.c_uint64)]),
    "echokv_prefill_attention": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_int, C.c_void_p,
                                           C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p, C.c_uint64,
                                           C.c_void_p]),
    "echokv_layer_step_host": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p]),
    "echokv_get_device_status": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32)]),
    "echokv_launch_count": (C.c_int64, [C.c_void_p]),
    "echokv_decode_path": (C.c_int, [C.c_void_p]),
    "echokv_set_decode_path": (C.c_int, [C.c_void_p, C.c_int]),
    "echokv_side_buffer_bytes": (C.c_int, [C.POINTER(echokv_config), C.c_int, C.c_int, C.POINTER(C.c_uint64)]),
    "echokv_set_full_precision_window": (C.c_int, [C.c_void_p, C.c_int, C.c_int, C.POINTER(C.c_void_p),
                                                   C.POINTER(C.c_void_p)]),
    "echokv_rope_table_bytes": (C.c_int, [C.POINTER(echokv_config), C.POINTER(C.c_uint64)]),
    "echokv_set_rope": (C.c_int, [C.c_void_p, C.c_double, C.c_void_p, C.c_uint64, C.c_void_p]),
    "echokv_rope_enabled": (C.c_int, [C.c_void_p]),
    "echokv_absorbed_workspace_bytes": (C.c_int, [C.POINTER(echokv_config), C.POINTER(C.c_uint64)]),
    "echokv_enable_absorbed": (C.c_int, [C.c_void_p, C.c_void_p, C.c_uint64]),
    "echokv_decode_mode": (C.c_int, [C.c_void_p]),
    "echokv_set_decode_mode": (C.c_int, [C.c_void_p, C.c_int]),
    "echokv_stored_path": (C.c_int, [C.c_void_p]),
    "echokv_set_stored_path": (C.c_int, [C.c_void_p, C.c_int]),
    "echokv_set_kernel_timing": (C.c_int, [C.c_void_p, C.c_int]),
    "echokv_read_kernel_timing": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "echokv_read_kernel_timing_by_kind": (C.c_int, [C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_int64)]),
    "echokv_diag_bounded_wait": (C.c_int, [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]),
    "echokv_diag_page_order": (C.c_int, [C.c_void_p, C.POINTER(C.c_int32)]),
    "echokv_full_attention_noalloc": (C.c_int, [C.POINTER(echokv_config), C.c_void_p, C.c_void_p, C.c_void_p,
                                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p, C.c_int,
                                                C.c_void_p, C.c_void_p]),
    "echokv_noalloc_scratch_bytes": (C.c_uint64, []),
    "echokv_strerror": (C.c_char_p, [C.c_int]),
}

_lib = None


def lib() -> C.CDLL:
    """The loaded shared library (loaded once)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError("libechokv.so is not built: run `python -m paper_2603_22910_b200.build` "
                               "(there is no fallback implementation)")
        _lib = C.CDLL(LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(_lib, name)
            fn.restype = res
            fn.argtypes = args
    return _lib


class EchoKVError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (%d)" % (where, echokv_strerror(status), status))


def echokv_strerror(status: int) -> str:
    return lib().echokv_strerror(status).decode()


def _check(status: int, where: str) -> None:
    if status != ECHOKV_OK:
        raise EchoKVError(status, where)


def _ptr(t) -> int | None:
    """Device / host address of a torch tensor (None stays NULL)."""
    return None if t is None else t.data_ptr()


def _stream_handle(stream) -> int | None:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream or None


def make_config(*, n_layers, n_q_heads, n_kv_heads, head_dim, group_size, n_retained_heads,
                page_tokens, max_batch, max_pages_per_seq, n_pages, dtype, softmax_scale=0.0,
                device=0, n_retained_dims=0, save_k=0) -> echokv_config:
    return echokv_config(n_layers, n_q_heads, n_kv_heads, head_dim, group_size, n_retained_heads,
                         page_tokens, max_batch, max_pages_per_seq, dtype, n_pages, softmax_scale, device,
                         n_retained_dims, save_k)


def echokv_query_sizes(cfg: echokv_config) -> echokv_sizes:
    out = echokv_sizes()
    _check(lib().echokv_query_sizes(C.byref(cfg), C.byref(out)), "echokv_query_sizes")
    return out


class Context:
    """A context plus the torch tensors it borrows (pools, workspace, block table).

    Allocation is the only thing done here that is not a direct C-ABI call.
    """

    def __init__(self, cfg: echokv_config, zero_pools: bool = False):
        import torch
        self.torch = torch
        self.cfg = cfg
        self.device = torch.device("cuda", cfg.device)
        self.sizes = echokv_query_sizes(cfg)
        self.tdtype = torch.bfloat16 if cfg.dtype == ECHOKV_BF16 else torch.float32
        D = cfg.n_kv_heads * cfg.head_dim
        m = cfg.n_retained_dims if cfg.n_retained_dims else cfg.n_retained_heads * cfg.head_dim
        self.D, self.m = D, m
        alloc = torch.zeros if zero_pools else torch.empty
        self.k_pools, self.v_pools = [], []
        self.mk = D if (cfg.save_k and m < D) else m      # K dims a compressed layer stores ("save K": all of them)
        for l in range(cfg.n_layers):
            for pools, width in ((self.k_pools, D if l % cfg.group_size == 0 else self.mk),
                                 (self.v_pools, D if l % cfg.group_size == 0 else m)):
                if width == 0:
                    pools.append(None)
                else:
                    pools.append(alloc((cfg.n_pages, cfg.page_tokens, width), dtype=self.tdtype, device=self.device))
        self.workspace = torch.empty(self.sizes.workspace_bytes, dtype=torch.uint8, device=self.device)
        self.block_table = torch.zeros((cfg.max_batch, cfg.max_pages_per_seq), dtype=torch.int32,
                                       device=self.device)
        n = cfg.n_layers
        self._kp = (C.c_void_p * n)(*[_ptr(t) for t in self.k_pools])
        self._vp = (C.c_void_p * n)(*[_ptr(t) for t in self.v_pools])
        buf = echokv_buffers(C.cast(self._kp, C.POINTER(C.c_void_p)), C.cast(self._vp, C.POINTER(C.c_void_p)),
                             self.workspace.data_ptr(), self.sizes.workspace_bytes)
        self.handle = C.c_void_p()
        _check(lib().echokv_create(C.byref(cfg), C.byref(buf), C.byref(self.handle)), "echokv_create")
        _check(lib().echokv_set_block_table(self.handle, self.block_table.data_ptr()), "echokv_set_block_table")
        self._weights = {}

    # -- direct wrappers -------------------------------------------------------------
    def close(self):
        if self.handle:
            lib().echokv_destroy(self.handle)
            self.handle = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_block_table(self, table) -> None:
        """Copy a host/device int32 table into the borrowed device block table."""
        self.block_table[:table.shape[0], :table.shape[1]].copy_(table)

    def set_weights(self, layer: int, Wk, Wv, bk=None, bv=None) -> None:
        self._weights[layer] = (Wk, Wv, bk, bv)   # keep the borrowed tensors alive
        _check(lib().echokv_set_weights(self.handle, layer, _ptr(Wk), _ptr(Wv), _ptr(bk), _ptr(bv)),
               "echokv_set_weights")

    def append_kv(self, layer: int, k_new, v_new, positions, seq_slots=None, stream=None) -> None:
        _check(lib().echokv_append_kv(self.handle, layer, _ptr(k_new), _ptr(v_new), _ptr(seq_slots),
                                      _ptr(positions), k_new.shape[0], _stream_handle(stream)),
               "echokv_append_kv")

    def append_kv_chunk(self, layer: int, k_new, v_new, first_positions, seq_slots=None, stream=None) -> None:
        """k_new, v_new [B][n_tokens][H_kv][d]: n_tokens consecutive new tokens per sequence."""
        _check(lib().echokv_append_kv_chunk(self.handle, layer, _ptr(k_new), _ptr(v_new), _ptr(seq_slots),
                                            _ptr(first_positions), k_new.shape[1], k_new.shape[0],
                                            _stream_handle(stream)), "echokv_append_kv_chunk")

    def compress_layer(self, layer: int, k_full, v_full, seq_lens, seq_begins=None, seq_slots=None, stream=None) -> None:
        """Evict a layer cached at full width ([n_pages][page_tokens][D] pools) down to its retained dims."""
        _check(lib().echokv_compress_layer(self.handle, layer, _ptr(k_full), _ptr(v_full), _ptr(seq_slots),
                                           _ptr(seq_begins), _ptr(seq_lens), seq_lens.shape[0],
                                           _stream_handle(stream)), "echokv_compress_layer")

    def decode_attention(self, layer: int, q, seq_lens, out=None, seq_slots=None, stream=None):
        out = self._out(q) if out is None else out
        _check(lib().echokv_decode_attention(self.handle, layer, _ptr(q), _ptr(out), _ptr(seq_slots),
                                             _ptr(seq_lens), q.shape[0], _stream_handle(stream)),
               "echokv_decode_attention")
        return out

    def prefill_attention(self, layer: int, q, seq_lens, out=None, seq_slots=None, stream=None, k_recent=None,
                          v_recent=None):
        """q [B][n_q][H_q][d]: the last n_q cached tokens of every sequence as causal queries.  The scratch
        for the rebuilt cache rows is allocated on first use and kept.  k_recent, v_recent [B][n_q + n_window - 1][D]:
        whole K / V rows of the chunk and the n_window - 1 tokens before it (needed while a window is set)."""
        if getattr(self, "prefill_scratch", None) is None:
            n = C.c_uint64(0)
            _check(lib().echokv_prefill_scratch_bytes(C.byref(self.cfg), C.byref(n)), "echokv_prefill_scratch_bytes")
            self.prefill_scratch = self.torch.empty(n.value, dtype=self.torch.uint8, device=self.device)
        out = self._out(q) if out is None else out
        _check(lib().echokv_prefill_attention(self.handle, layer, _ptr(q), _ptr(out), q.shape[1], _ptr(seq_slots),
                                              _ptr(seq_lens), q.shape[0], _ptr(k_recent), _ptr(v_recent),
                                              self.prefill_scratch.data_ptr(),
                                              self.prefill_scratch.numel(), _stream_handle(stream)),
               "echokv_prefill_attention")
        return out

    def full_attention(self, layer: int, q, seq_lens, out=None, seq_slots=None, stream=None):
        out = self._out(q) if out is None else out
        _check(lib().echokv_full_attention(self.handle, layer, _ptr(q), _ptr(out), _ptr(seq_slots),
                                           _ptr(seq_lens), q.shape[0], _stream_handle(stream)),
               "echokv_full_attention")
        return out

    def layer_step_host(self, layer: int, q_host, k_new_host, v_new_host, out_host, seq_lens_host,
                        attend: bool = True, stream=None) -> None:
        _check(lib().echokv_layer_step_host(self.handle, layer, _ptr(q_host), _ptr(k_new_host),
                                            _ptr(v_new_host), _ptr(out_host), _ptr(seq_lens_host),
                                            k_new_host.shape[0], 1 if attend else 0,
                                            _stream_handle(stream)),
               "echokv_layer_step_host")

    def device_status(self) -> int:
        v = C.c_int32(0)
        _check(lib().echokv_get_device_status(self.handle, C.byref(v)), "echokv_get_device_status")
        return v.value

    def launch_count(self) -> int:
        return lib().echokv_launch_count(self.handle)

    def decode_path(self) -> int:
        return lib().echokv_decode_path(self.handle)

    def diag_page_order(self) -> int:
        out = C.c_int32(-1)
        _check(lib().echokv_diag_page_order(self.handle, C.byref(out)), "echokv_diag_page_order")
        return out.value

    def set_decode_path(self, path: int) -> None:
        _check(lib().echokv_set_decode_path(self.handle, path), "echokv_set_decode_path")

    def set_full_precision_window(self, n_sink: int, n_window: int) -> None:
        """Keep the first n_sink and the last n_window tokens of every sequence uncompressed: allocates the
        side buffers of the compressed layers ([max_batch][n_sink + n_window][D - m]) and hands them over."""
        cfg, n = self.cfg, self.cfg.n_layers
        self.k_side, self.v_side = [], []
        for l in range(n):
            if l % cfg.group_size == 0 or self.D == self.m or n_sink + n_window == 0:
                self.k_side.append(None)
                self.v_side.append(None)
            else:
                shape = (cfg.max_batch, n_sink + n_window, self.D - self.m)
                self.k_side.append(self.torch.zeros(shape, dtype=self.tdtype, device=self.device))
                self.v_side.append(self.torch.zeros(shape, dtype=self.tdtype, device=self.device))
        self._ks = (C.c_void_p * n)(*[_ptr(t) for t in self.k_side])
        self._vs = (C.c_void_p * n)(*[_ptr(t) for t in self.v_side])
        _check(lib().echokv_set_full_precision_window(self.handle, n_sink, n_window,
                                                      C.cast(self._ks, C.POINTER(C.c_void_p)),
                                                      C.cast(self._vs, C.POINTER(C.c_void_p))),
               "echokv_set_full_precision_window")
        self.n_sink, self.n_window = n_sink, n_window

    def set_rope(self, theta: float, stream=None) -> None:
        """Rotate cached keys to their positions when they are read (the cache holds un-rotated keys):
        allocates the (cos, sin) table and has the library fill it.  theta = 0 switches it off."""
        if not theta:
            _check(lib().echokv_set_rope(self.handle, 0.0, None, 0, None), "echokv_set_rope")
            self.rope_table = None
            return
        n = C.c_uint64(0)
        _check(lib().echokv_rope_table_bytes(C.byref(self.cfg), C.byref(n)), "echokv_rope_table_bytes")
        self.rope_table = self.torch.empty(n.value, dtype=self.torch.uint8, device=self.device)
        _check(lib().echokv_set_rope(self.handle, float(theta), self.rope_table.data_ptr(), n.value,
                                     _stream_handle(stream)), "echokv_set_rope")

    def rope_enabled(self) -> bool:
        return bool(lib().echokv_rope_enabled(self.handle))

    def enable_absorbed(self) -> None:
        """Allocate the absorbed mode's workspace and switch the context to that mode."""
        n = C.c_uint64(0)
        _check(lib().echokv_absorbed_workspace_bytes(C.byref(self.cfg), C.byref(n)), "echokv_absorbed_workspace_bytes")
        self.workspace_absorbed = self.torch.empty(n.value, dtype=self.torch.uint8, device=self.device)
        _check(lib().echokv_enable_absorbed(self.handle, self.workspace_absorbed.data_ptr(), n.value),
               "echokv_enable_absorbed")

    def decode_mode(self) -> int:
        return lib().echokv_decode_mode(self.handle)

    def set_decode_mode(self, mode: int) -> None:
        _check(lib().echokv_set_decode_mode(self.handle, mode), "echokv_set_decode_mode")

    def stored_path(self) -> int:
        return lib().echokv_stored_path(self.handle)

    def set_stored_path(self, path: int) -> None:
        _check(lib().echokv_set_stored_path(self.handle, path), "echokv_set_stored_path")

    def set_kernel_timing(self, enable: bool) -> None:
        _check(lib().echokv_set_kernel_timing(self.handle, 1 if enable else 0), "echokv_set_kernel_timing")

    def read_kernel_timing(self):
        """(total milliseconds, launches) of the dominant kernel since the last read."""
        ms, n = C.c_double(0.0), C.c_int64(0)
        _check(lib().echokv_read_kernel_timing(self.handle, C.byref(ms), C.byref(n)), "echokv_read_kernel_timing")
        return ms.value, n.value

    def read_kernel_timing_by_kind(self):
        """{"stored": (ms, launches), "recon": (ms, launches)} since the last read."""
        ms, n = (C.c_double * 4)(), (C.c_int64 * 4)()
        _check(lib().echokv_read_kernel_timing_by_kind(self.handle, ms, n), "echokv_read_kernel_timing_by_kind")
        return {"stored": (ms[0], n[0]), "recon": (ms[1], n[1]), "absorb_k": (ms[2], n[2]), "absorb_v": (ms[3], n[3])}

    def diag_bounded_wait(self, limit_cycles: int, stream=None):
        """Run the bounded-wait probe; returns the device tensor int32[2] saying how its two warps left."""
        left = self.torch.zeros(2, dtype=self.torch.int32, device=self.device)
        _check(lib().echokv_diag_bounded_wait(self.handle, int(limit_cycles), left.data_ptr(), _stream_handle(stream)),
               "echokv_diag_bounded_wait")
        return left

    def _out(self, q):
        return self.torch.empty(q.shape, dtype=self.torch.float32, device=self.device)


def echokv_full_attention_noalloc(cfg: echokv_config, k_pool, v_pool, block_table, q, out, seq_lens,
                                  seq_slots=None, status_out=None, stream=None) -> None:
    """Full-cache attention without a context or a workspace, for callers that cannot allocate
    device memory: partial results live in a fixed 8 MiB array inside the library.  Tensors are
    only read for their addresses; nothing is allocated here either.  Calls sharing a device must
    not overlap on the GPU, and the first call on a device should precede any stream capture."""
    _check(lib().echokv_full_attention_noalloc(C.byref(cfg), _ptr(k_pool), _ptr(v_pool), _ptr(block_table),
                                               _ptr(q), _ptr(out), _ptr(seq_slots), _ptr(seq_lens),
                                               q.shape[0], _ptr(status_out), _stream_handle(stream)),
           "echokv_full_attention_noalloc")


def config_for(w, n_pages: int | None = None, device: int = 0, max_batch: int | None = None) -> echokv_config:
    """echokv_config of a synth.Workload."""
    pages = w.pages_per_seq
    return make_config(n_layers=w.n_layers, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                       head_dim=w.head_dim, group_size=w.group_size,
                       n_retained_heads=w.n_retained_heads, page_tokens=w.page_tokens,
                       max_batch=max_batch or w.batch, max_pages_per_seq=pages,
                       n_pages=n_pages or w.batch * pages,
                       dtype=ECHOKV_BF16 if w.dtype == "bf16" else ECHOKV_FP32,
                       softmax_scale=1.0 / math.sqrt(w.head_dim), device=device,
                       n_retained_dims=w.n_retained_dims, save_k=1 if w.save_k else 0)
