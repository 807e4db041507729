"""ctypes wrapper around the CPU oracle (kl_oracle.c).

TEST INFRASTRUCTURE ONLY: nothing on the product path may import this module.
It defines the expected result of a decode step (Sections 1-2 of the paper name
the blocks; the arithmetic is written out in kl_oracle.c).  The wrapper adds no
arithmetic: it marshals numpy buffers and loops over layers and sequences.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "kl_oracle.c"
_LIB = _HERE / "libkl_oracle.so"


def build(force: bool = False) -> Path:
    """Compile kl_oracle.c with gcc (OpenMP over independent rows / heads only)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".so.tmp{os.getpid()}")
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", str(tmp), str(_SRC), "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Desc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in
                ("n_layers", "hidden", "n_q_heads", "n_kv_heads", "head_dim", "ffn", "vocab", "max_ctx")] + \
               [("rms_eps", C.c_double), ("rope_theta", C.c_double)]


class Counters(C.Structure):
    _fields_ = [(n, C.c_uint64) for n in ("macs", "weight_bytes", "embed_bytes", "kv_read_bytes", "kv_write_bytes")]

    def as_dict(self) -> dict:
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "norm1", "norm2",
                                           "bq", "bk", "bv")] + \
               [("n_experts", C.c_int32), ("top_k", C.c_int32), ("router", C.c_void_p),   # mixture-of-experts layers
                ("ex_gate", C.POINTER(C.c_void_p)), ("ex_up", C.POINTER(C.c_void_p)), ("ex_down", C.POINTER(C.c_void_p))]
DENSE_FIELDS = ("wq", "wk", "wv", "wo", "wgate", "wup", "wdown", "norm1", "norm2", "bq", "bk", "bv")


_lib = None


def lib():
    global _lib
    if _lib is None:
        l = C.CDLL(str(build()))
        dp, vp, cp = C.POINTER(C.c_double), C.c_void_p, C.POINTER(Counters)
        l.ko_bf16_to_double.restype = C.c_double
        l.ko_bf16_to_double.argtypes = [C.c_uint16]
        l.ko_bf16_rne.restype = C.c_uint16
        l.ko_bf16_rne.argtypes = [C.c_double]
        l.ko_matvec.argtypes = [vp, C.c_int, C.c_int, dp, dp, cp, C.c_int]
        l.ko_matvec.restype = None
        l.ko_rmsnorm.argtypes = [dp, vp, C.c_int, C.c_double, dp, cp, C.c_int]
        l.ko_rmsnorm.restype = None
        l.ko_rope.argtypes = [dp, C.c_int, C.c_int, C.c_double]
        l.ko_rope.restype = None
        l.ko_softmax.argtypes = [dp, C.c_int, dp]
        l.ko_softmax.restype = None
        l.ko_silu.argtypes = [C.c_double]
        l.ko_silu.restype = C.c_double
        l.ko_attention_head.argtypes = [dp, vp, vp, C.c_int, C.c_int, C.c_size_t, dp, dp]
        l.ko_attention_head.restype = None
        l.ko_embed.argtypes = [C.POINTER(Desc), vp, C.c_int, dp, cp, C.c_int]
        l.ko_embed.restype = None
        l.ko_decoder_layer.argtypes = [C.POINTER(Desc), C.POINTER(LayerWeights), vp, vp, C.c_int, dp, cp, C.c_int]
        l.ko_decoder_layer.restype = C.c_int
        l.ko_classifier.argtypes = [C.POINTER(Desc), vp, vp, dp, dp, cp, C.c_int]
        l.ko_classifier.restype = C.c_int
        l.ko_moe_route.argtypes = [dp, C.c_int, C.c_int, C.POINTER(C.c_int32), dp]
        l.ko_moe_route.restype = None
        l.ko_argmax.argtypes = [dp, C.c_int]
        l.ko_argmax.restype = C.c_int
        l.ko_num_threads.restype = C.c_int
        _lib = l
    return _lib


def num_threads() -> int:
    return int(lib().ko_num_threads())


def as_u16(a) -> np.ndarray:
    """bf16 payload as a contiguous numpy uint16 array (accepts numpy uint16 or a CPU torch bf16 tensor)."""
    if isinstance(a, np.ndarray):
        assert a.dtype == np.uint16
        return np.ascontiguousarray(a)
    import torch  # buffers only
    assert a.dtype == torch.bfloat16 and a.device.type == "cpu"
    return a.contiguous().view(torch.uint16).numpy()


def _dp(a: np.ndarray):
    assert a.dtype == np.float64 and a.flags.c_contiguous
    return a.ctypes.data_as(C.POINTER(C.c_double))


def _vp(a: np.ndarray):
    assert a.flags.c_contiguous
    return C.c_void_p(a.ctypes.data)


def make_desc(shape, max_ctx: int) -> Desc:
    """`shape` is any object with the ModelShape attribute names."""
    return Desc(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim, shape.ffn,
                shape.vocab, max_ctx, float(shape.rms_eps), float(shape.rope_theta))


# ------------------------------------------------------------------ operator-level entry points (for the pins)

def bf16_to_double(u16) -> np.ndarray:
    u = np.asarray(u16, dtype=np.uint16)
    with np.errstate(invalid="ignore"):
        return (u.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def bf16_rne(v) -> np.ndarray:
    v = np.asarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.uint16)
    f = lib().ko_bf16_rne
    flat_in, flat_out = v.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = f(float(flat_in[i]))
    return out


def matvec(W_u16: np.ndarray, x: np.ndarray) -> np.ndarray:
    W = as_u16(W_u16)
    R, K = W.shape
    x = np.ascontiguousarray(x, dtype=np.float64)
    y = np.empty(R, dtype=np.float64)
    lib().ko_matvec(_vp(W), R, K, _dp(x), _dp(y), None, 0)
    return y


def rmsnorm(x: np.ndarray, g_u16: np.ndarray, eps: float) -> np.ndarray:
    x = np.ascontiguousarray(x, dtype=np.float64)
    g = as_u16(g_u16)
    y = np.empty_like(x)
    lib().ko_rmsnorm(_dp(x), _vp(g), x.size, eps, _dp(y), None, 0)
    return y


def rope(u: np.ndarray, p: int, theta: float) -> np.ndarray:
    out = np.ascontiguousarray(u, dtype=np.float64).copy()
    lib().ko_rope(_dp(out), out.size, int(p), float(theta))
    return out


def softmax(s: np.ndarray) -> np.ndarray:
    s = np.ascontiguousarray(s, dtype=np.float64)
    w = np.empty_like(s)
    lib().ko_softmax(_dp(s), s.size, _dp(w))
    return w


def silu(z: float) -> float:
    return float(lib().ko_silu(float(z)))


def attention_head(q: np.ndarray, K_u16: np.ndarray, V_u16: np.ndarray) -> np.ndarray:
    """q[hd] against K,V [n][hd] bf16."""
    K, V = as_u16(K_u16), as_u16(V_u16)
    n, hd = K.shape
    q = np.ascontiguousarray(q, dtype=np.float64)
    out = np.empty(hd, dtype=np.float64)
    scratch = np.empty(2 * n, dtype=np.float64)
    lib().ko_attention_head(_dp(q), _vp(K), _vp(V), n, hd, hd, _dp(out), _dp(scratch))
    return out


def moe_route(logits: np.ndarray, k: int):
    """Chosen experts (descending logit, lower index first among equals) and their softmax weights."""
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    idx = (C.c_int32 * k)()
    w = np.empty(k, dtype=np.float64)
    lib().ko_moe_route(_dp(logits), logits.size, k, idx, _dp(w))
    return list(idx), w


def argmax(logits: np.ndarray) -> int:
    logits = np.ascontiguousarray(logits, dtype=np.float64)
    return int(lib().ko_argmax(_dp(logits), logits.size))


# ------------------------------------------------------------------ block-level driver

class Oracle:
    """Decode steps of one model, one sequence at a time, with optional layer streaming.

    layer_weights(l) -> dict name -> bf16 buffer for layer l (wq wk wv wo wgate wup wdown norm1 norm2, and
    bq bk bv for decoders whose q, k, v projections carry a bias);
    globals_: dict with 'norm_f', 'lm_head' and either 'embed' (the table) or a callable
    'embed_row'(token) -> bf16 row.
    """

    def __init__(self, shape, max_ctx: int, layer_weights, globals_):
        self.shape = shape
        self.desc = make_desc(shape, max_ctx)
        self.max_ctx = max_ctx
        self._layer_weights = layer_weights
        self._globals = globals_
        self.counters = Counters()

    def _layer_struct(self, l: int):
        w = self._layer_weights(l)
        keep = {k: as_u16(v) for k, v in w.items()}
        s = LayerWeights()
        for n in DENSE_FIELDS:
            if n in keep:
                setattr(s, n, keep[n].ctypes.data)
        E = int(getattr(self.shape, "n_experts", 0) or 0)
        if E > 0:   # tensors router, wgate_e<i>, wup_e<i>, wdown_e<i>
            s.n_experts, s.top_k = E, int(self.shape.top_k)
            s.router = keep["router"].ctypes.data
            for field, stem in (("ex_gate", "wgate_e"), ("ex_up", "wup_e"), ("ex_down", "wdown_e")):
                arr = (C.c_void_p * E)(*[keep[f"{stem}{e}"].ctypes.data for e in range(E)])
                keep["_" + field] = arr
                setattr(s, field, C.cast(arr, C.POINTER(C.c_void_p)))
        return s, keep

    def embed(self, token: int) -> np.ndarray:
        x = np.empty(self.shape.hidden, dtype=np.float64)
        if "embed" in self._globals:
            E = as_u16(self._globals["embed"])
            lib().ko_embed(C.byref(self.desc), _vp(E), int(token), _dp(x), C.byref(self.counters), 0)
        else:
            row = as_u16(self._globals["embed_row"](int(token)))
            lib().ko_embed(C.byref(self.desc), _vp(row), 0, _dp(x), C.byref(self.counters), 0)
        return x

    def step(self, kv_cache_u16: np.ndarray, tokens, positions, layers=None, want_logits: bool = True):
        """One decode step for every sequence b.  kv_cache_u16: [L][2][B][nkv][max_ctx][hd] uint16, updated in place.

        Returns (hidden [B,H], logits [B,V] or None, next_tokens [B] or None).
        `layers` restricts the decoder blocks run (default: all) -- used for bounded timing samples.
        """
        s = self.shape
        B = len(tokens)
        assert kv_cache_u16.dtype == np.uint16 and kv_cache_u16.flags.c_contiguous
        assert kv_cache_u16.shape == (s.n_layers, 2, B, s.n_kv_heads, self.max_ctx, s.head_dim)
        xs = [self.embed(int(t)) for t in tokens]
        for l in (range(s.n_layers) if layers is None else layers):
            ws, keep = self._layer_struct(l)
            for b in range(B):
                kc, vc = kv_cache_u16[l, 0, b], kv_cache_u16[l, 1, b]
                rc = lib().ko_decoder_layer(C.byref(self.desc), C.byref(ws), _vp(kc), _vp(vc), int(positions[b]),
                                            _dp(xs[b]), C.byref(self.counters), 0)
                if rc != 0:
                    raise RuntimeError("ko_decoder_layer rejected its arguments")
            del keep
        hidden = np.stack(xs)
        if not want_logits:
            return hidden, None, None
        logits = np.empty((B, s.vocab), dtype=np.float64)
        gf, wlm = as_u16(self._globals["norm_f"]), as_u16(self._globals["lm_head"])
        for b in range(B):
            rc = lib().ko_classifier(C.byref(self.desc), _vp(gf), _vp(wlm), _dp(xs[b]), _dp(logits[b]),
                                     C.byref(self.counters), 0)
            if rc != 0:
                raise RuntimeError("ko_classifier failed")
        nxt = np.array([argmax(logits[b]) for b in range(B)], dtype=np.int32)
        return hidden, logits, nxt


def count_step(shape, batch: int, position: int, max_ctx: int | None = None) -> dict:
    """Run the oracle's own loops in count-only mode: MACs and bytes of one decode step at `position`
    for `batch` identical-length sequences (parameters are counted once, KV and MACs per sequence)."""
    max_ctx = max_ctx or position + 1
    d = make_desc(shape, max_ctx)
    total = Counters()
    for b in range(batch):
        c = Counters()
        lib().ko_embed(C.byref(d), None, 0, None, C.byref(c), 1)
        lw = LayerWeights()
        lw.n_experts, lw.top_k = int(getattr(shape, "n_experts", 0) or 0), int(getattr(shape, "top_k", 0) or 0)
        for _ in range(shape.n_layers):
            rc = lib().ko_decoder_layer(C.byref(d), C.byref(lw), None, None, position, None, C.byref(c), 1)
            assert rc == 0
        lib().ko_classifier(C.byref(d), None, None, None, None, C.byref(c), 1)
        total.macs += c.macs
        total.embed_bytes += c.embed_bytes
        total.kv_read_bytes += c.kv_read_bytes
        total.kv_write_bytes += c.kv_write_bytes
        if b == 0:
            total.weight_bytes = c.weight_bytes  # parameters are read once per step, whatever the batch
    return total.as_dict()
