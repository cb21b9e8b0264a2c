"""The C-ABI library: it loads, exports every symbol the header declares, and rejects bad
arguments on the host before touching a device (no compute calls here)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_1905_05686_b200 import build
    build.build()
    from paper_1905_05686_b200 import binding
    return binding


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lrbi.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"LRBI_API[^;(]*?\b(lrbi_\w+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert len(names) >= 17 and "lrbi_decode_mask" in names and "lrbi_masked_gemm" in names
    L = ctypes.CDLL(lib.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n


def test_size_helpers_follow_the_packed_format(lib):
    from paper_1905_05686_b200 import synth
    for name in synth.CONFIG_ORDER:
        c = synth.CONFIGS[name]
        lay = lib.Layout.of(c)
        gr, gc = c.grid
        assert lib.lib().lrbi_packed_ip_words(ctypes.byref(lay)) == gr * gc * c.tile_rows * c.kw
        assert lib.lib().lrbi_packed_iz_words(ctypes.byref(lay)) == gr * gc * c.tile_cols * c.kw
        assert lib.lib().lrbi_mask_words(ctypes.byref(lay)) == c.mask_words
    bad = lib.Layout(0, 5, 1, 1, 1)
    assert lib.lib().lrbi_mask_words(ctypes.byref(bad)) == 0


def test_argument_errors_are_reported_without_a_launch(lib):
    L = lib.lib()
    lay = lib.Layout(64, 64, 32, 32, 4)
    before = lib.launch_count()
    p = ctypes.c_void_p(0x1000)           # never dereferenced: the checks fail first
    null = ctypes.c_void_p(0)
    assert L.lrbi_decode_mask(ctypes.byref(lay), null, p, p, 0, null) == lib.ERR_INVALID_ARG
    assert L.lrbi_decode_mask(ctypes.byref(lay), p, p, ctypes.c_void_p(0x1004), 0, null) == lib.ERR_INVALID_ARG   # misaligned
    assert L.lrbi_decode_mask(ctypes.byref(lay), p, p, p, 99, null) == lib.ERR_INVALID_ARG
    bad = lib.Layout(64, 64, 32, 32, 0)   # rank 0
    assert L.lrbi_decode_mask(ctypes.byref(bad), p, p, p, 0, null) == lib.ERR_INVALID_ARG
    assert L.lrbi_masked_gemm(ctypes.byref(lay), p, p, p, p, 0, p, 0, 0, null) == lib.ERR_INVALID_ARG      # batch 0
    assert L.lrbi_masked_gemm(ctypes.byref(lay), p, p, p, p, 4, p, 7, 0, null) == lib.ERR_INVALID_ARG      # dtype
    assert L.lrbi_masked_gemm(ctypes.byref(lay), p, p, null, p, 4, p, 0, 0, null) == lib.ERR_INVALID_ARG
    odd = lib.Layout(64, 63, 32, 32, 4)   # cols % 8 != 0: the vector kernels refuse, nothing is launched
    assert L.lrbi_masked_gemm(ctypes.byref(odd), p, p, p, p, 4, p, 0, lib.ALGO_GEMV, null) == lib.ERR_UNSUPPORTED
    assert L.lrbi_masked_gemm(ctypes.byref(odd), p, p, p, p, 64, p, 0, lib.ALGO_TENSOR, null) == lib.ERR_UNSUPPORTED
    assert lib.launch_count() == before
    assert lib.status_string(lib.ERR_UNSUPPORTED)


def test_kernel_choice_per_config(lib):
    from paper_1905_05686_b200 import synth
    c = synth.CONFIGS["alexnet_fc"]
    assert lib.masked_gemm_choice(c, 1) == lib.ALGO_GEMV
    assert lib.masked_gemm_choice(c, 16) == lib.ALGO_TENSOR
    assert lib.masked_gemm_choice(synth.CONFIGS["ffn_16384x4096"], 4096) == lib.ALGO_TENSOR
    assert lib.masked_gemm_choice(synth.Layer("odd", 37, 45, 16, 20, 7, 0.2), 5) == lib.ALGO_GENERIC


def test_plan_query_runs_without_a_device(lib):
    """The plan is host arithmetic: which instantiation of the tensor-core kernel a call would run."""
    from paper_1905_05686_b200 import synth
    p = lib.masked_gemm_plan(synth.CONFIGS["ffn_16384x4096"], 4096)
    assert (p.algo, p.cta_pair, p.batch_tile, p.panel_columns, p.k_splits) == (lib.ALGO_TENSOR, 1, 512, 256, 1)
    assert p.scratch_bytes == 0 and p.stages >= 3
    p = lib.masked_gemm_plan(synth.CONFIGS["ffn_16384x4096"], 4096, lib.ALGO_TENSOR_PAIR)
    assert (p.cta_pair, p.batch_tile) == (1, 256)
    p = lib.masked_gemm_plan(synth.CONFIGS["alexnet_fc"], 16)
    assert p.algo == lib.ALGO_TENSOR and p.cta_pair == 0 and p.k_splits > 1
    assert p.scratch_bytes == p.k_splits * 16 * 4096 * 4
    assert lib.masked_gemm_static_bytes(synth.CONFIGS["alexnet_fc"], 16) == p.scratch_bytes
    p = lib.masked_gemm_plan(synth.CONFIGS["alexnet_fc"], 1)
    assert p.algo == lib.ALGO_GEMV and p.k_splits == 1
    with pytest.raises(lib.LrbiError) as e:
        lib.masked_gemm_plan(synth.Layer("odd", 37, 45, 16, 20, 7, 0.2), 64, lib.ALGO_TENSOR)
    assert e.value.code == lib.ERR_UNSUPPORTED
