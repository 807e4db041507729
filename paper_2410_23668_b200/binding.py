"""Thin ctypes binding of libkl.so: the same names as include/kl.h, argument marshalling only.

PyTorch appears here for device memory and streams alone (arenas, KV cache, token / logit buffers); every step
of the decode path runs inside the library's kernels.  There is no fallback: if the library is missing this
module raises at load time.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

_LIB_PATH = Path(__file__).resolve().parent / "libkl.so"

KL_OK = 0
KL_ERR_INVALID_ARG = -1
KL_ERR_UNSUPPORTED_SHAPE = -2
KL_ERR_NOT_LOADED = -3
KL_ERR_CUDA = -4
KL_ERR_SYNC_TIMEOUT = -5
KL_ERR_OUT_OF_RANGE = -6
KL_ERR_TOO_LARGE = -7
KL_STATIC_ARGMAX_MAX_BATCH = 256
KL_MODE_LOOPED = 0
KL_MODE_PER_LAYER = 1
KL_MODE_PER_STAGE = 2

TENSOR_IDS = {"embed": 0, "wq": 1, "wk": 2, "wv": 3, "wo": 4, "wgate": 5, "wup": 6, "wdown": 7,
              "norm1": 8, "norm2": 9, "norm_f": 10, "lm_head": 11, "bq": 12, "bk": 13, "bv": 14, "router": 15}
KL_FLAG_QKV_BIAS = 1
KL_FLAG_NO_STASH = 2

# every symbol include/kl.h declares
EXPORTS = ("kl_workspace_bytes", "kl_create", "kl_load_weights", "kl_kv_cache_bytes", "kl_set_mode", "kl_decode_step",
           "kl_decode_step_host", "kl_argmax_advance", "kl_read_hidden", "kl_last_status", "kl_launch_count",
           "kl_set_wait_limit_ns", "kl_debug_skip_signal_once", "kl_status_string", "kl_destroy", "kl_profile_enable",
           "kl_profile_read", "kl_set_trace", "kl_set_tensor_core_attention", "kl_stash_mode", "kl_argmax_advance_static", "kl_set_batched_path",
           "kl_set_dependent_launch", "kl_decode_greedy_host", "kl_decode_greedy", "kl_decode_greedy_tokens",
           "kl_decode_greedy_tokens_host", "kl_debug_set_step", "kl_debug_set_jitter", "kl_load_expert_weights")


class ModelDesc(C.Structure):
    _fields_ = [("n_layers", C.c_uint32), ("hidden", C.c_uint32), ("n_q_heads", C.c_uint32),
                ("n_kv_heads", C.c_uint32), ("head_dim", C.c_uint32), ("ffn", C.c_uint32), ("vocab", C.c_uint32),
                ("rms_eps", C.c_float), ("rope_theta", C.c_float), ("max_batch", C.c_uint32),
                ("max_ctx", C.c_uint32), ("flags", C.c_uint32), ("n_experts", C.c_uint32), ("top_k", C.c_uint32)]


_lib = None


def lib():
    """Loads libkl.so (built in-tree by paper_2410_23668_b200.build / __graft_entry__.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2410_23668_b200.build` "
                           "(there is no CPU or PyTorch fallback for the decode path)")
    l = C.CDLL(str(_LIB_PATH))
    vp, u32, i32 = C.c_void_p, C.c_uint32, C.c_int32
    l.kl_workspace_bytes.argtypes = [C.POINTER(ModelDesc), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    l.kl_workspace_bytes.restype = i32
    l.kl_create.argtypes = [C.POINTER(ModelDesc), vp, vp, C.POINTER(vp)]
    l.kl_create.restype = i32
    l.kl_load_weights.argtypes = [vp, C.c_int, C.c_int, vp, C.c_size_t, vp]
    l.kl_load_weights.restype = i32
    l.kl_load_expert_weights.argtypes = [vp, C.c_int, C.c_int, C.c_int, vp, C.c_size_t, vp]
    l.kl_load_expert_weights.restype = i32
    l.kl_kv_cache_bytes.argtypes = [vp, u32]
    l.kl_kv_cache_bytes.restype = C.c_size_t
    l.kl_set_mode.argtypes = [vp, C.c_int]
    l.kl_set_mode.restype = i32
    l.kl_decode_step.argtypes = [vp, vp, vp, vp, vp, u32, vp]
    l.kl_decode_step.restype = i32
    l.kl_decode_step_host.argtypes = [vp, vp, vp, vp, vp, u32, vp]
    l.kl_decode_step_host.restype = i32
    l.kl_decode_greedy_host.argtypes = [vp, vp, vp, vp, vp, u32, vp]
    l.kl_decode_greedy_host.restype = i32
    l.kl_decode_greedy.argtypes = [vp, vp, vp, vp, vp, u32, C.c_int, vp]
    l.kl_decode_greedy.restype = i32
    l.kl_decode_greedy_tokens.argtypes = [vp, vp, vp, vp, vp, vp, u32, u32, C.c_int, vp]
    l.kl_decode_greedy_tokens.restype = i32
    l.kl_decode_greedy_tokens_host.argtypes = [vp, i32, i32, vp, vp, u32, vp]
    l.kl_decode_greedy_tokens_host.restype = i32
    l.kl_argmax_advance.argtypes = [vp, vp, vp, vp, u32, vp]
    l.kl_argmax_advance.restype = i32
    l.kl_argmax_advance_static.argtypes = [vp, u32, vp, vp, u32, vp]
    l.kl_argmax_advance_static.restype = i32
    l.kl_read_hidden.argtypes = [vp, vp, u32, vp]
    l.kl_read_hidden.restype = i32
    l.kl_last_status.argtypes = [vp]
    l.kl_last_status.restype = i32
    l.kl_launch_count.argtypes = [vp]
    l.kl_launch_count.restype = C.c_uint64
    l.kl_set_wait_limit_ns.argtypes = [vp, C.c_uint64]
    l.kl_set_wait_limit_ns.restype = i32
    l.kl_debug_skip_signal_once.argtypes = [vp, C.c_int]
    l.kl_debug_skip_signal_once.restype = i32
    l.kl_debug_set_jitter.argtypes = [vp, u32, u32]
    l.kl_debug_set_jitter.restype = i32
    l.kl_debug_set_step.argtypes = [vp, u32, C.POINTER(u32)]
    l.kl_debug_set_step.restype = i32
    l.kl_profile_enable.argtypes = [vp, u32]
    l.kl_profile_enable.restype = i32
    l.kl_profile_read.argtypes = [vp, C.POINTER(u32), C.POINTER(C.c_float), C.POINTER(C.c_float)]
    l.kl_profile_read.restype = i32
    l.kl_set_trace.argtypes = [vp, vp, C.POINTER(u32), C.POINTER(u32), C.POINTER(u32)]
    l.kl_set_trace.restype = i32
    l.kl_set_tensor_core_attention.argtypes = [vp, C.c_int]
    l.kl_set_tensor_core_attention.restype = i32
    l.kl_stash_mode.argtypes = [vp]
    l.kl_stash_mode.restype = C.c_int
    l.kl_set_batched_path.argtypes = [vp, C.c_int]
    l.kl_set_batched_path.restype = i32
    l.kl_set_dependent_launch.argtypes = [vp, C.c_int]
    l.kl_set_dependent_launch.restype = i32
    l.kl_status_string.argtypes = [i32]
    l.kl_status_string.restype = C.c_char_p
    l.kl_destroy.argtypes = [vp]
    l.kl_destroy.restype = None
    _lib = l
    return l


class KlError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {kl_status_string(code)} ({code})")


def kl_status_string(code: int) -> str:
    return lib().kl_status_string(code).decode()


def _check(code: int, where: str) -> None:
    if code != KL_OK:
        raise KlError(code, where)


def make_desc(shape, max_batch: int, max_ctx: int, stash: bool = True) -> ModelDesc:
    return ModelDesc(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                     shape.vocab, float(shape.rms_eps), float(shape.rope_theta), max_batch, max_ctx,
                     (KL_FLAG_QKV_BIAS if getattr(shape, "qkv_bias", False) else 0) | (0 if stash else KL_FLAG_NO_STASH),
                     int(getattr(shape, "n_experts", 0) or 0), int(getattr(shape, "top_k", 0) or 0))


def kl_workspace_bytes(desc: ModelDesc) -> tuple[int, int]:
    w, s = C.c_size_t(), C.c_size_t()
    _check(lib().kl_workspace_bytes(C.byref(desc), C.byref(w), C.byref(s)), "kl_workspace_bytes")
    return w.value, s.value


def _ptr(t) -> int:
    return 0 if t is None else int(t.data_ptr())


def _stream_ptr(stream) -> int:
    return 0 if stream is None else int(stream.cuda_stream)


def kl_argmax_advance_static(logits_d, tokens_d, positions_d, batch: int, stream=None) -> None:
    """Sampling block without a handle: scratch in a fixed array inside the library, nothing is allocated."""
    _check(lib().kl_argmax_advance_static(_ptr(logits_d), int(logits_d.shape[-1]), _ptr(tokens_d), _ptr(positions_d), batch,
                                          _stream_ptr(stream)), "kl_argmax_advance_static")


class Decoder:
    """One model instance on the current CUDA device.  Owns the two arenas as torch uint8 tensors."""

    def __init__(self, shape, max_batch: int, max_ctx: int, device="cuda", stash: bool = True):
        import torch
        self.torch = torch
        self.shape = shape
        self.max_batch, self.max_ctx = max_batch, max_ctx
        self.desc = make_desc(shape, max_batch, max_ctx, stash)
        wb, sb = kl_workspace_bytes(self.desc)
        self.weight_bytes, self.scratch_bytes = wb, sb
        self.weight_arena = torch.empty(wb, dtype=torch.uint8, device=device)
        self.scratch_arena = torch.empty(sb, dtype=torch.uint8, device=device)
        h = C.c_void_p()
        _check(lib().kl_create(C.byref(self.desc), _ptr(self.weight_arena), _ptr(self.scratch_arena), C.byref(h)), "kl_create")
        self.handle = h

    def close(self) -> None:
        if getattr(self, "handle", None):
            lib().kl_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C-ABI calls, same names
    def kl_load_weights(self, name: str, layer: int, tensor, stream=None) -> None:
        t = tensor.contiguous()
        assert t.dtype == self.torch.bfloat16
        if "_e" in name:   # an expert's matrix of a mixture-of-experts layer: wgate_e<i>, wup_e<i>, wdown_e<i>
            stem, expert = name.rsplit("_e", 1)
            _check(lib().kl_load_expert_weights(self.handle, TENSOR_IDS[stem], layer, int(expert), _ptr(t), t.numel() * 2,
                                                _stream_ptr(stream)), f"kl_load_expert_weights({name}, {layer})")
        else:
            _check(lib().kl_load_weights(self.handle, TENSOR_IDS[name], layer, _ptr(t), t.numel() * 2, _stream_ptr(stream)),
                   f"kl_load_weights({name}, {layer})")
        if t.device.type == "cpu":
            self.torch.cuda.synchronize()  # pageable source must outlive the copy

    def kl_kv_cache_bytes(self, batch: int) -> int:
        return int(lib().kl_kv_cache_bytes(self.handle, batch))

    def kl_set_mode(self, mode: int) -> None:
        _check(lib().kl_set_mode(self.handle, mode), "kl_set_mode")

    def kl_decode_step(self, tokens_d, positions_d, kv_cache_d, logits_d, batch: int, stream=None) -> None:
        _check(lib().kl_decode_step(self.handle, _ptr(tokens_d), _ptr(positions_d), _ptr(kv_cache_d), _ptr(logits_d),
                                    batch, _stream_ptr(stream)), "kl_decode_step")

    def kl_decode_step_host(self, tokens_h, positions_h, kv_cache_d, logits_h, batch: int, stream=None) -> None:
        _check(lib().kl_decode_step_host(self.handle, _ptr(tokens_h), _ptr(positions_h), _ptr(kv_cache_d),
                                         _ptr(logits_h), batch, _stream_ptr(stream)), "kl_decode_step_host")

    def kl_decode_greedy(self, tokens_d, positions_d, kv_cache_d, logits_d, batch: int, restart: bool, stream=None) -> None:
        _check(lib().kl_decode_greedy(self.handle, _ptr(tokens_d), _ptr(positions_d), _ptr(kv_cache_d), _ptr(logits_d),
                                      batch, 1 if restart else 0, _stream_ptr(stream)), "kl_decode_greedy")

    def kl_decode_greedy_tokens(self, tokens_d, positions_d, kv_cache_d, logits_d, out_tokens_d, n_tokens: int, batch: int,
                                restart: bool, stream=None) -> None:
        _check(lib().kl_decode_greedy_tokens(self.handle, _ptr(tokens_d), _ptr(positions_d), _ptr(kv_cache_d), _ptr(logits_d),
                                             _ptr(out_tokens_d), n_tokens, batch, 1 if restart else 0, _stream_ptr(stream)),
               "kl_decode_greedy_tokens")

    def kl_decode_greedy_tokens_host(self, token: int, position: int, kv_cache_d, out_tokens_h, n_tokens: int, stream=None) -> None:
        _check(lib().kl_decode_greedy_tokens_host(self.handle, token, position, _ptr(kv_cache_d), _ptr(out_tokens_h), n_tokens,
                                                  _stream_ptr(stream)), "kl_decode_greedy_tokens_host")

    def kl_decode_greedy_host(self, tokens_h, positions_h, kv_cache_d, next_tokens_h, batch: int, stream=None) -> None:
        _check(lib().kl_decode_greedy_host(self.handle, _ptr(tokens_h), _ptr(positions_h), _ptr(kv_cache_d),
                                           _ptr(next_tokens_h), batch, _stream_ptr(stream)), "kl_decode_greedy_host")

    def kl_argmax_advance(self, logits_d, tokens_d, positions_d, batch: int, stream=None) -> None:
        _check(lib().kl_argmax_advance(self.handle, _ptr(logits_d), _ptr(tokens_d), _ptr(positions_d), batch,
                                       _stream_ptr(stream)), "kl_argmax_advance")

    def kl_read_hidden(self, hidden_d, batch: int, stream=None) -> None:
        _check(lib().kl_read_hidden(self.handle, _ptr(hidden_d), batch, _stream_ptr(stream)), "kl_read_hidden")

    def kl_last_status(self) -> int:
        return int(lib().kl_last_status(self.handle))

    def kl_launch_count(self) -> int:
        return int(lib().kl_launch_count(self.handle))

    def kl_profile_enable(self, capacity: int) -> None:
        _check(lib().kl_profile_enable(self.handle, capacity), "kl_profile_enable")

    def kl_profile_read(self, n: int) -> tuple[list[float], list[float]]:
        cnt = C.c_uint32(n)
        dec, cls = (C.c_float * n)(), (C.c_float * n)()
        _check(lib().kl_profile_read(self.handle, C.byref(cnt), dec, cls), "kl_profile_read")
        return list(dec[:cnt.value]), list(cls[:cnt.value])

    def kl_set_trace(self, trace_d=None) -> tuple[int, int, int]:
        a, b, c = C.c_uint32(), C.c_uint32(), C.c_uint32()
        _check(lib().kl_set_trace(self.handle, _ptr(trace_d), C.byref(a), C.byref(b), C.byref(c)), "kl_set_trace")
        return a.value, b.value, c.value

    def kl_stash_mode(self) -> int:
        return int(lib().kl_stash_mode(self.handle))

    def kl_set_tensor_core_attention(self, on: bool) -> None:
        _check(lib().kl_set_tensor_core_attention(self.handle, 1 if on else 0), "kl_set_tensor_core_attention")

    def kl_set_batched_path(self, on: bool) -> None:
        _check(lib().kl_set_batched_path(self.handle, 1 if on else 0), "kl_set_batched_path")

    def kl_set_dependent_launch(self, on: bool) -> None:
        _check(lib().kl_set_dependent_launch(self.handle, 1 if on else 0), "kl_set_dependent_launch")

    def kl_set_wait_limit_ns(self, ns: int) -> None:
        _check(lib().kl_set_wait_limit_ns(self.handle, ns), "kl_set_wait_limit_ns")

    def kl_debug_skip_signal_once(self, stage: int) -> None:
        _check(lib().kl_debug_skip_signal_once(self.handle, stage), "kl_debug_skip_signal_once")

    def kl_debug_set_jitter(self, seed: int, max_ns: int) -> None:
        _check(lib().kl_debug_set_jitter(self.handle, seed, max_ns), "kl_debug_set_jitter")

    def kl_debug_set_step(self, step: int | None = None) -> int:
        """Sets the step counter behind the tags (None: only queries); returns the step number at which it wraps."""
        w = C.c_uint32()
        _check(lib().kl_debug_set_step(self.handle, 0xffffffff if step is None else step, C.byref(w)), "kl_debug_set_step")
        return w.value

    # -- marshalling helpers
    def load_model(self, layer_weights, globals_, stream=None) -> None:
        """layer_weights(l) -> dict of bf16 tensors; globals_: dict with embed, norm_f, lm_head."""
        for l in range(self.shape.n_layers):
            for name, t in layer_weights(l).items():
                self.kl_load_weights(name, l, t, stream)
        for name in ("embed", "norm_f", "lm_head"):
            self.kl_load_weights(name, -1, globals_[name], stream)
        self.torch.cuda.synchronize()
