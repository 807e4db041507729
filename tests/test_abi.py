"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol include/kl.h declares.
Host-side argument validation is exercised too (no kernel runs here)."""
import ctypes as C
import re
from pathlib import Path

import pytest

from paper_2410_23668_b200 import binding, build, inputs as gen

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module")
def lib():
    build.build_library()
    return binding.lib()


def test_every_declared_symbol_is_exported(lib):
    header = (ROOT / "include" / "kl.h").read_text()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(kl_[a-z_0-9]+)\s*\(", header))
    assert declared == set(binding.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_status_strings(lib):
    assert binding.kl_status_string(0) == "KL_OK"
    assert binding.kl_status_string(-5) == "KL_ERR_SYNC_TIMEOUT"
    assert binding.kl_status_string(-99) == "KL_ERR_UNKNOWN"


def test_workspace_sizes_and_shape_validation(lib):
    d = binding.make_desc(gen.LLAMA31_8B, 1, 4096 + 256)
    wb, sb = binding.kl_workspace_bytes(d)
    s = gen.LLAMA31_8B
    per_layer = s.hidden * s.head_dim * (2 * s.n_q_heads + 2 * s.n_kv_heads) + 3 * s.hidden * s.ffn + 2 * s.hidden
    tensors = 2 * (s.n_layers * per_layer + s.hidden + 2 * s.vocab * s.hidden)
    assert tensors <= wb <= tensors + 64 * 1024  # the arena is the tensors plus alignment padding only
    assert sb < 8 << 20
    # unsupported shapes are refused, not mangled
    bad = binding.make_desc(gen.ModelShape(2, 100, 4, 2, 64, 512, 1000), 1, 64)  # hidden not a multiple of 8
    w, sc = C.c_size_t(), C.c_size_t()
    assert lib.kl_workspace_bytes(C.byref(bad), C.byref(w), C.byref(sc)) == binding.KL_ERR_UNSUPPORTED_SHAPE
    bad = binding.make_desc(gen.ModelShape(2, 128, 6, 4, 64, 512, 1000), 1, 64)  # heads not divisible
    assert lib.kl_workspace_bytes(C.byref(bad), C.byref(w), C.byref(sc)) == binding.KL_ERR_UNSUPPORTED_SHAPE
    assert lib.kl_workspace_bytes(None, C.byref(w), C.byref(sc)) == binding.KL_ERR_INVALID_ARG
    # group sizes: three query heads per kv head only where the tensor-core attention loop exists (head size 64 / 128)
    ok = binding.make_desc(gen.ModelShape(2, 3072, 24, 8, 128, 8192, 1000), 1, 64)
    assert lib.kl_workspace_bytes(C.byref(ok), C.byref(w), C.byref(sc)) == binding.KL_OK
    bad = binding.make_desc(gen.ModelShape(2, 768, 24, 8, 32, 1024, 1000), 1, 64)
    assert lib.kl_workspace_bytes(C.byref(bad), C.byref(w), C.byref(sc)) == binding.KL_ERR_UNSUPPORTED_SHAPE
    # flags: the projection biases add their vectors to every layer; unknown flags are refused
    import dataclasses
    sb_shape = dataclasses.replace(s, qkv_bias=True)
    wb2, _ = binding.kl_workspace_bytes(binding.make_desc(sb_shape, 1, 4096 + 256))
    qr = s.q_dim + 2 * s.kv_dim
    assert s.n_layers * qr * 2 <= wb2 - wb <= s.n_layers * (qr * 2 + 256)
    bad = binding.make_desc(s, 1, 64)
    bad.flags = 4   # not a flag of the interface (1: biases, 2: no stash mode)
    assert lib.kl_workspace_bytes(C.byref(bad), C.byref(w), C.byref(sc)) == binding.KL_ERR_UNSUPPORTED_SHAPE
    # a batched handle (max_batch > 1) carries the operand, partial-result and attention buffers of the batched path
    _, sb32 = binding.kl_workspace_bytes(binding.make_desc(s, 32, 4096 + 256))
    assert sb < sb32 < 256 << 20


def test_null_handle_calls_are_rejected(lib):
    assert lib.kl_set_mode(None, 0) == binding.KL_ERR_INVALID_ARG
    assert lib.kl_decode_step(None, None, None, None, None, 1, None) == binding.KL_ERR_INVALID_ARG
    assert lib.kl_last_status(None) == binding.KL_ERR_INVALID_ARG
    assert lib.kl_decode_greedy(None, None, None, None, None, 1, 1, None) == binding.KL_ERR_INVALID_ARG
    assert lib.kl_decode_greedy_tokens(None, None, None, None, None, None, 4, 1, 1, None) == binding.KL_ERR_INVALID_ARG
    assert lib.kl_decode_greedy_tokens_host(None, 0, 0, None, None, 4, None) == binding.KL_ERR_INVALID_ARG
    assert lib.kl_kv_cache_bytes(None, 1) == 0
    assert lib.kl_launch_count(None) == 0
    lib.kl_destroy(None)
