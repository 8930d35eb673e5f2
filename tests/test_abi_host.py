"""C-ABI checks that need no GPU: the library loads, exports every symbol the header
declares, sizes are right, and argument errors come back as status codes."""
import ctypes as C
import os
import re

import pytest

from paper_2603_22910_b200 import binding, build, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    build.build()
    return binding.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "echokv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(echokv_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(lib):
    names = declared_symbols()
    assert len(names) >= 14
    for n in names:
        assert hasattr(lib, n), "library does not export " + n
        assert n in binding.EXPORTS, "binding lacks " + n
    assert sorted(binding.EXPORTS) == names


def test_query_sizes_c1(lib):
    w = synth.C1
    cfg = binding.config_for(w)
    s = binding.echokv_query_sizes(cfg)
    rows = w.batch * w.pages_per_seq * w.page_tokens
    assert s.anchor_pool_bytes == rows * w.D * 2
    assert s.compressed_pool_bytes == rows * w.m * 2
    assert s.block_table_bytes == w.batch * w.pages_per_seq * 4
    assert s.max_partials == w.context // 128 + 1  # one partial per 128 tokens, one for sink / window tokens
    part = w.batch * w.n_q_heads * s.max_partials
    assert s.workspace_bytes >= part * (8 + 4 * w.head_dim)
    w0 = synth.C0
    s0 = binding.echokv_query_sizes(binding.config_for(w0))
    assert s0.max_partials == w0.context // 64 + 1
    assert s0.anchor_pool_bytes == w0.context * w0.D * 4


@pytest.mark.parametrize("field,value,code", [
    ("n_layers", 0, binding.ECHOKV_EINVAL), ("n_kv_heads", 3, binding.ECHOKV_EINVAL),
    ("n_retained_heads", 9, binding.ECHOKV_EINVAL), ("n_retained_heads", -1, binding.ECHOKV_EINVAL),
    ("head_dim", 96, binding.ECHOKV_EUNSUPPORTED), ("page_tokens", 24, binding.ECHOKV_EUNSUPPORTED),
    ("dtype", 7, binding.ECHOKV_EINVAL), ("group_size", 0, binding.ECHOKV_EINVAL),
    ("softmax_scale", -1.0, binding.ECHOKV_EINVAL), ("n_pages", 0, binding.ECHOKV_EINVAL),
])
def test_bad_configs_are_rejected(lib, field, value, code):
    cfg = binding.config_for(synth.C0)
    setattr(cfg, field, value)
    out = binding.echokv_sizes()
    assert lib.echokv_query_sizes(C.byref(cfg), C.byref(out)) == code
    with pytest.raises(binding.EchoKVError):
        binding.echokv_query_sizes(cfg)


def test_null_arguments_return_einval(lib):
    cfg = binding.config_for(synth.C0)
    assert lib.echokv_query_sizes(None, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_query_sizes(C.byref(cfg), None) == binding.ECHOKV_EINVAL
    h = C.c_void_p()
    assert lib.echokv_create(C.byref(cfg), None, C.byref(h)) == binding.ECHOKV_EINVAL
    assert lib.echokv_create(C.byref(cfg), None, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_block_table(None, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_weights(None, 0, None, None, None, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_append_kv(None, 0, None, None, None, None, 1, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_decode_attention(None, 0, None, None, None, None, 1, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_full_attention(None, 0, None, None, None, None, 1, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_layer_step_host(None, 0, None, None, None, None, None, 1, 1, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_get_device_status(None, None) == binding.ECHOKV_EINVAL
    assert lib.echokv_set_decode_path(None, 1) == binding.ECHOKV_EINVAL
    assert lib.echokv_launch_count(None) == 0 and lib.echokv_decode_path(None) == 0
    lib.echokv_destroy(None)


def test_create_checks_buffers_before_touching_cuda(lib):
    cfg = binding.config_for(synth.C0)
    sizes = binding.echokv_query_sizes(cfg)
    n = cfg.n_layers
    fake = (C.c_void_p * n)(*[0x1000] * n)
    h = C.c_void_p()
    small = binding.echokv_buffers(C.cast(fake, C.POINTER(C.c_void_p)), C.cast(fake, C.POINTER(C.c_void_p)),
                                   0x10000, sizes.workspace_bytes - 1)
    assert lib.echokv_create(C.byref(cfg), C.byref(small), C.byref(h)) == binding.ECHOKV_ECAPACITY
    misaligned = binding.echokv_buffers(C.cast(fake, C.POINTER(C.c_void_p)), C.cast(fake, C.POINTER(C.c_void_p)),
                                        0x10008, sizes.workspace_bytes)
    assert lib.echokv_create(C.byref(cfg), C.byref(misaligned), C.byref(h)) == binding.ECHOKV_EINVAL
    nulls = (C.c_void_p * n)(*[None] * n)
    nopool = binding.echokv_buffers(C.cast(nulls, C.POINTER(C.c_void_p)), C.cast(nulls, C.POINTER(C.c_void_p)),
                                    0x10000, sizes.workspace_bytes)
    assert lib.echokv_create(C.byref(cfg), C.byref(nopool), C.byref(h)) == binding.ECHOKV_EINVAL
    assert not h.value


def test_strerror_names_every_code(lib):
    seen = set()
    for code in range(0, -13, -1):
        s = binding.echokv_strerror(code)
        assert s and s != "unknown status"
        seen.add(s)
    assert len(seen) == 13
    assert binding.echokv_strerror(-99) == "unknown status"


def test_no_fallback_when_library_is_missing(monkeypatch, tmp_path):
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError, match="no fallback"):
        binding.lib()
