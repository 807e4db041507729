"""Pins for the CPU oracle: every part of it is checked against something that is not the oracle --
closed forms, invariants, brute force in pure Python, a re-statement with torch CPU library operators,
and the figures the paper prints (operation-intensity table, kernel-call counts)."""
import csv
import math
from pathlib import Path

import numpy as np
import pytest
import dataclasses

import torch

from oracle import kl_oracle as ko
from paper_2410_23668_b200 import inputs as gen

GOLDEN = Path(__file__).parent / "golden"

SHAPES = {
    "8B": gen.LLAMA31_8B,
    "70B": gen.LLAMA31_70B,
    "405B": gen.ModelShape(126, 16384, 128, 8, 128, 53248, 128256, 1e-5, 500000.0),
}


def u16(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.uint16).numpy()


def bf16_of(a) -> np.ndarray:
    """float array -> bf16 payload via torch's own rounding (inputs are chosen float-exact)."""
    return u16(torch.tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16))


# ------------------------------------------------------------------ bf16 conversions

def test_bf16_roundtrip_and_ties():
    # decode: every one of the 65536 payloads agrees with torch's bf16 -> float
    allp = np.arange(65536, dtype=np.uint16)
    ref = torch.from_numpy(allp.copy()).view(torch.bfloat16).to(torch.float64).numpy()
    got = ko.bf16_to_double(allp)
    fin = np.isfinite(ref)
    assert np.array_equal(got[fin], ref[fin])
    # encode: exact bf16 values are fixed points
    some = allp[fin][::97]
    assert np.array_equal(ko.bf16_rne(ko.bf16_to_double(some)), some)
    # ties go to the even mantissa: 1 + 2^-8 is halfway between 1.0 (even) and 1 + 2^-7 (odd)
    assert ko.bf16_rne([1.0 + 2.0 ** -8])[0] == 0x3F80
    assert ko.bf16_rne([1.0 + 2.0 ** -7 + 2.0 ** -8])[0] == 0x3F82  # halfway between ...81 (odd) and ...82 (even)
    assert ko.bf16_rne([-(1.0 + 2.0 ** -8)])[0] == 0xBF80
    # just above / below a tie (only resolvable in double): must not double-round through float
    assert ko.bf16_rne([1.0 + 2.0 ** -8 + 2.0 ** -40])[0] == 0x3F81
    assert ko.bf16_rne([1.0 + 2.0 ** -8 - 2.0 ** -40])[0] == 0x3F80
    # random floats: same as torch float32 -> bf16 (round to nearest even)
    rng = np.random.default_rng(0)
    v = (rng.standard_normal(2000) * 10 ** rng.uniform(-3, 3, 2000)).astype(np.float32)
    assert np.array_equal(ko.bf16_rne(v.astype(np.float64)), bf16_of(v))
    assert ko.bf16_rne([0.0])[0] == 0


# ------------------------------------------------------------------ operators

def test_matvec_identity_and_transpose_sensitivity():
    K = 24
    eye = bf16_of(np.eye(K))
    x = np.random.default_rng(1).standard_normal(K)
    assert np.array_equal(ko.matvec(eye, x), x)
    # a non-symmetric 0/1 matrix catches a transposed operand: y = W x with W[r, (r+1)%K] = 1 is a rotation
    W = np.zeros((K, K), dtype=np.float32)
    for r in range(K):
        W[r, (r + 1) % K] = 1.0
    assert np.array_equal(ko.matvec(bf16_of(W), x), np.roll(x, -1))
    # rectangular, against numpy float64 on the decoded values
    Wr = np.random.default_rng(2).standard_normal((7, 40)).astype(np.float32)
    Wb = bf16_of(Wr)
    x2 = np.random.default_rng(3).standard_normal(40)
    assert np.allclose(ko.matvec(Wb, x2), ko.bf16_to_double(Wb) @ x2, rtol=1e-13, atol=1e-13)


def test_rmsnorm_unit_rms_scale_invariance_and_eps():
    H = 64
    x = np.random.default_rng(4).standard_normal(H) * 3.0
    ones = bf16_of(np.ones(H))
    y = ko.rmsnorm(x, ones, 0.0)
    assert abs(math.sqrt(np.mean(y * y)) - 1.0) < 1e-12
    # scale invariance (eps = 0)
    assert np.allclose(ko.rmsnorm(7.5 * x, ones, 0.0), y, rtol=1e-12)
    # eps sits inside the root, added to the MEAN of squares: x = c * ones gives c / sqrt(c^2 + eps)
    c, eps = 0.01, 1e-5
    y2 = ko.rmsnorm(np.full(H, c), ones, eps)
    assert np.allclose(y2, c / math.sqrt(c * c + eps), rtol=1e-13)
    # gain multiplies after normalisation
    g = bf16_of(np.linspace(0.5, 2.0, H))
    assert np.allclose(ko.rmsnorm(x, g, 0.0), y * ko.bf16_to_double(g), rtol=1e-13)


def test_rope_norm_identity_relative_and_pairing():
    hd, theta = 16, 10000.0
    rng = np.random.default_rng(5)
    q, k = rng.standard_normal(hd), rng.standard_normal(hd)
    assert np.array_equal(ko.rope(q, 0, theta), q)  # position 0 is the identity
    for p in (1, 7, 4096, 65535):
        assert abs(np.linalg.norm(ko.rope(q, p, theta)) - np.linalg.norm(q)) < 1e-9 * np.linalg.norm(q)
    # the score of a rotated pair depends only on the distance m - n
    d1 = ko.rope(q, 100, theta) @ ko.rope(k, 90, theta)
    d2 = ko.rope(q, 1010, theta) @ ko.rope(k, 1000, theta)
    assert abs(d1 - d2) < 1e-9
    # half-split pairing with frequency theta^(-2i/hd): the unit vector e_i rotates into the (i, i+hd/2) plane
    for i in (0, 3, hd // 2 - 1):
        e = np.zeros(hd)
        e[i] = 1.0
        r = ko.rope(e, 5, theta)
        ang = 5.0 * theta ** (-2.0 * i / hd)
        expect = np.zeros(hd)
        expect[i], expect[i + hd // 2] = math.cos(ang), math.sin(ang)
        assert np.allclose(r, expect, atol=1e-12)
    # same rotation written with complex numbers (independent formulation)
    p = 1234
    z = (q[: hd // 2] + 1j * q[hd // 2:]) * np.exp(1j * p * theta ** (-2.0 * np.arange(hd // 2) / hd))
    assert np.allclose(ko.rope(q, p, theta), np.concatenate([z.real, z.imag]), atol=1e-9)


def test_softmax_rows_sum_to_one_shift_invariant_uniform():
    rng = np.random.default_rng(6)
    s = rng.standard_normal(300) * 20
    w = ko.softmax(s)
    assert abs(w.sum() - 1.0) < 1e-12 and (w >= 0).all()
    assert np.allclose(ko.softmax(s + 1000.0), w, rtol=1e-10)
    assert np.allclose(ko.softmax(np.full(17, 3.25)), 1.0 / 17, rtol=1e-14)
    # closed form on two entries: softmax([a, b])[0] = 1 / (1 + e^(b-a))
    assert abs(ko.softmax(np.array([0.3, 1.7]))[0] - 1.0 / (1.0 + math.exp(1.4))) < 1e-15
    # no overflow for large scores
    assert np.isfinite(ko.softmax(np.array([1e4, 1e4 - 1.0]))).all()


def test_silu_values():
    assert ko.silu(0.0) == 0.0
    assert abs(ko.silu(40.0) - 40.0) < 1e-12
    assert abs(ko.silu(-40.0)) < 1e-12
    assert abs(ko.silu(1.0) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-15
    assert abs(ko.silu(-2.0) + 2.0 / (1.0 + math.exp(2.0))) < 1e-15


def test_argmax_lowest_index_on_ties():
    """Sampling block: the largest logit wins, and among equal maxima the LOWEST index (a rule that takes the last
    of them, i.e. `>=` in place of `>`, fails the first three cases)."""
    assert ko.argmax(np.array([0.5, 3.0, -1.0, 3.0, 2.0, 3.0])) == 1          # maximum at 1, 3 and 5
    assert ko.argmax(np.array([7.0, 7.0, 7.0, 7.0])) == 0                       # all equal
    assert ko.argmax(np.array([-2.0, -1.0, -1.0])) == 1                         # negative values, tie at the end
    assert ko.argmax(np.array([1.0, 2.0, 5.0])) == 2                            # no tie, maximum last
    assert ko.argmax(np.array([-0.0, 0.0])) == 0                                # signed zeros compare equal
    rng = np.random.default_rng(0)
    for _ in range(50):                                                         # against numpy's first-maximum rule
        v = rng.integers(-3, 4, size=40).astype(np.float64)
        assert ko.argmax(v) == int(np.argmax(v))


def test_attention_brute_force_and_special_cases():
    rng = np.random.default_rng(7)
    n, hd = 7, 8
    q = rng.standard_normal(hd)
    Kf = rng.standard_normal((n, hd)).astype(np.float32)
    Vf = rng.standard_normal((n, hd)).astype(np.float32)
    Kb, Vb = bf16_of(Kf), bf16_of(Vf)
    Kd, Vd = ko.bf16_to_double(Kb), ko.bf16_to_double(Vb)
    # brute force, pure Python
    s = [sum(q[d] * Kd[j][d] for d in range(hd)) / math.sqrt(hd) for j in range(n)]
    m = max(s)
    e = [math.exp(v - m) for v in s]
    z = sum(e)
    ref = [sum(e[j] / z * Vd[j][d] for j in range(n)) for d in range(hd)]
    got = ko.attention_head(q, Kb, Vb)
    assert np.allclose(got, ref, rtol=1e-12, atol=1e-14)
    # all keys equal -> plain mean of V
    Ke = bf16_of(np.tile(Kf[0], (n, 1)))
    assert np.allclose(ko.attention_head(q, Ke, Vb), Vd.mean(axis=0), rtol=1e-12)
    # a single position -> its value row, whatever the score
    assert np.allclose(ko.attention_head(q, Kb[:1], Vb[:1]), Vd[0], rtol=1e-14)
    # 1/sqrt(hd) scale: one-hot q and K rows that differ only in that coordinate -> closed-form weights
    q1 = np.zeros(hd)
    q1[2] = 4.0
    K2 = np.zeros((2, hd), dtype=np.float32)
    K2[1, 2] = 1.0
    V2 = np.zeros((2, hd), dtype=np.float32)
    V2[1, :] = 1.0
    w1 = 1.0 / (1.0 + math.exp(-4.0 / math.sqrt(hd)))
    assert np.allclose(ko.attention_head(q1, bf16_of(K2), bf16_of(V2)), w1, rtol=1e-13)


# ------------------------------------------------------------------ whole blocks

def _tiny_setup(max_ctx=160, context=128, seed=0, shape=gen.TINY):
    layers = [gen.make_layer(shape, l, seed) for l in range(shape.n_layers)]
    glob = gen.make_globals(shape, seed)
    cache = gen.make_kv_cache(shape, 1, context, max_ctx, seed)
    return shape, layers, glob, cache


def test_gqa_head_mapping_constant_values():
    """Query head hq reads kv head hq div (nq/nkv).  Cached V of kv head g is the constant c_g and W_v = 0, so
    head hq outputs (1 - w_p) c_g with 0 < w_p < 1 the weight of the new (zero) value row: sign and bound of
    the output identify the kv head read.  W_o copies coordinate 0 of head hq into x[hq]; the MLP is off.
    An interleaved (hq mod nkv) or otherwise permuted grouping fails."""
    shape = gen.ModelShape(1, 32, 6, 3, 8, 16, 64, 1e-5, 10000.0)
    max_ctx, p = 12, 9
    rng = np.random.default_rng(8)
    G = shape.n_q_heads // shape.n_kv_heads
    consts = [0.5, -2.0, 3.0]
    cache = np.zeros(gen.kv_cache_shape(shape, 1, max_ctx), dtype=np.uint16)
    cache[0, 0] = bf16_of(rng.standard_normal((1, 3, max_ctx, 8)))  # random keys
    for g in range(3):
        cache[0, 1, 0, g] = bf16_of(np.full((max_ctx, 8), consts[g]))
    lw = {k: v.clone() for k, v in gen.make_layer(shape, 0, 3).items()}
    wo = np.zeros((shape.hidden, shape.q_dim), dtype=np.float32)
    for hq in range(6):
        wo[hq, hq * 8] = 1.0
    lw["wo"] = torch.tensor(wo).to(torch.bfloat16)
    lw["wv"] = torch.zeros_like(lw["wv"])
    lw["wgate"] = torch.zeros_like(lw["wgate"])
    orc = ko.Oracle(shape, max_ctx, lambda l: lw, gen.make_globals(shape, 3))
    x0 = orc.embed(5)
    hidden, _, _ = orc.step(cache, [5], [p], want_logits=False)
    delta = hidden[0][:6] - x0[:6]
    for hq in range(6):
        c = consts[hq // G]
        assert delta[hq] * c > 0 and abs(delta[hq]) < abs(c), "head %d does not read kv head %d" % (hq, hq // G)
    # heads of one group differ only through their weight on the zero row, so they stay within the same bound,
    # while the three groups are separated by sign / magnitude: group 1 is the only negative one
    assert (delta[2:4] < 0).all() and (delta[:2] > 0).all() and (delta[4:] > 0).all()
    # operator level, exact: constant V rows -> the output is that constant whatever the scores
    q = rng.standard_normal(8)
    out = ko.attention_head(q, cache[0, 0, 0, 1, :p], cache[0, 1, 0, 1, :p])
    assert np.allclose(out, consts[1], rtol=1e-14)


TINY_BIAS = dataclasses.replace(gen.TINY, qkv_bias=True)


def test_qkv_bias_against_torch_restatement_and_closed_form():
    """Decoders whose q, k, v projections carry a bias (the 72B decoder of Table 2).  (1) Four greedy steps agree with
    the torch restatement, which adds the bias with library operators (torch rounds the new cache row through
    float32, so a longer run eventually meets a double-rounding tie that differs by one bf16 step).  (2) W_q = W_k = W_v = 0: the cached rows are
    the biases themselves, v row = bf16(b_v) and k row = bf16(rope(b_k)) at every position -- a bias added after the
    rotation, to the wrong one of q / k / v, or dropped, fails.  (3) Zero biases give the bits of the model without
    biases."""
    shape, layers, glob, cache = _tiny_setup(shape=TINY_BIAS)
    assert all(n in layers[0] for n in ("bq", "bk", "bv"))
    orc = ko.Oracle(shape, cache.shape[4], lambda l: layers[l], glob)
    c_or, c_t = u16(cache).copy(), cache.clone()
    tok, p = int(gen.make_tokens(shape, 1, 0)[0]), 128
    for step in range(4):
        hidden, logits, nxt = orc.step(c_or, [tok], [p])
        h_ref, l_ref = _torch_reference_step(shape, layers, glob, c_t, tok, p)
        assert np.allclose(hidden[0], h_ref, rtol=1e-9, atol=1e-11), step
        assert np.allclose(logits[0], l_ref, rtol=1e-9, atol=1e-11), step
        c_t[:, :, :, :, p, :] = torch.from_numpy(c_or[:, :, :, :, p, :].copy()).view(torch.bfloat16)
        tok, p = int(nxt[0]), p + 1
    # (2)
    zl = [{k: v.clone() for k, v in lw.items()} for lw in layers]
    for lw in zl:
        for n in ("wq", "wk", "wv"):
            lw[n].zero_()
    c16 = u16(cache).copy()
    p = 131
    ko.Oracle(shape, cache.shape[4], lambda l: zl[l], glob).step(c16, [5], [p])
    hd, half = shape.head_dim, shape.head_dim // 2
    ang = p * shape.rope_theta ** (-2.0 * np.arange(half) / hd)
    for l in range(shape.n_layers):
        bv = zl[l]["bv"].to(torch.float64).numpy().reshape(shape.n_kv_heads, hd)
        assert np.array_equal(ko.bf16_to_double(c16[l, 1, 0, :, p, :]), bv)   # bf16 values: stored exactly
        bk = zl[l]["bk"].to(torch.float64).numpy().reshape(shape.n_kv_heads, hd)
        rot = np.concatenate([bk[:, :half] * np.cos(ang) - bk[:, half:] * np.sin(ang),
                              bk[:, half:] * np.cos(ang) + bk[:, :half] * np.sin(ang)], axis=1)
        assert np.allclose(ko.bf16_to_double(c16[l, 0, 0, :, p, :]), rot, rtol=2.0 ** -8, atol=1e-30)
    # (3)
    nb = [{k: (torch.zeros_like(v) if k in ("bq", "bk", "bv") else v) for k, v in lw.items()} for lw in layers]
    plain = [{k: v for k, v in lw.items() if k not in ("bq", "bk", "bv")} for lw in layers]
    ca, cb = u16(cache).copy(), u16(cache).copy()
    ha, la, _ = ko.Oracle(shape, cache.shape[4], lambda l: nb[l], glob).step(ca, [9], [128])
    hb, lb, _ = ko.Oracle(gen.TINY, cache.shape[4], lambda l: plain[l], glob).step(cb, [9], [128])
    assert np.array_equal(ha, hb) and np.array_equal(la, lb) and np.array_equal(ca, cb)


def test_zero_output_projections_pass_residual_through():
    """W_o = W_down = 0: x is unchanged by every layer, so logits = W_lm rmsnorm(E[tok]) in closed form,
    and the cache still receives bf16(rope(W_k a)) and bf16(W_v a)."""
    shape, layers, glob, cache = _tiny_setup()
    layers = [{k: v.clone() for k, v in lw.items()} for lw in layers]
    for lw in layers:
        lw["wo"].zero_()
        lw["wdown"].zero_()
    orc = ko.Oracle(shape, cache.shape[4], lambda l: layers[l], glob)
    tok, p = 77, 128
    c16 = u16(cache).copy()
    hidden, logits, nxt = orc.step(c16, [tok], [p])
    e = glob["embed"][tok].to(torch.float64).numpy()
    assert np.array_equal(hidden[0], e)
    a = e / math.sqrt(np.mean(e * e) + shape.rms_eps) * glob["norm_f"].to(torch.float64).numpy()
    ref_logits = glob["lm_head"].to(torch.float64).numpy() @ a
    assert np.allclose(logits[0], ref_logits, rtol=1e-12, atol=1e-14)
    assert nxt[0] == int(np.argmax(ref_logits))
    # cache row p of layer 0: V = bf16(W_v rmsnorm(e; g1)), K = bf16(rope(W_k rmsnorm(e; g1)))
    a1 = e / math.sqrt(np.mean(e * e) + shape.rms_eps) * layers[0]["norm1"].to(torch.float64).numpy()
    v = layers[0]["wv"].to(torch.float64).numpy() @ a1
    vrow = ko.bf16_to_double(c16[0, 1, 0, :, p, :]).reshape(-1)
    assert np.allclose(vrow, v, rtol=2.0 ** -8, atol=1e-30)  # within bf16 rounding
    k = (layers[0]["wk"].to(torch.float64).numpy() @ a1).reshape(shape.n_kv_heads, shape.head_dim)
    krow = ko.bf16_to_double(c16[0, 0, 0, :, p, :])
    for g in range(shape.n_kv_heads):
        assert abs(np.linalg.norm(krow[g]) - np.linalg.norm(k[g])) < 2.0 ** -7 * np.linalg.norm(k[g])
    # rows before p untouched, rows after p still zero
    assert np.array_equal(c16[:, :, :, :, :p], u16(cache)[:, :, :, :, :p])
    assert not c16[:, :, :, :, p + 1:].any()


def _torch_reference_step(shape, layers, glob, cache_bf16, token, p):
    """The same decode step written with torch CPU library operators in float64 (matmul,
    scaled_dot_product_attention, silu, complex multiplication for RoPE)."""
    F = torch.nn.functional
    f64 = torch.float64
    H, nq, nkv, hd = shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim
    x = glob["embed"][token].to(f64)
    rot = torch.polar(torch.ones(hd // 2, dtype=f64), p * shape.rope_theta ** (-2.0 * torch.arange(hd // 2, dtype=f64) / hd))

    def norm(v, g):
        return v * torch.rsqrt(v.pow(2).mean() + shape.rms_eps) * g.to(f64)

    def rope(u):  # u [heads, hd]
        z = torch.complex(u[:, : hd // 2], u[:, hd // 2:]) * rot
        return torch.cat([z.real, z.imag], dim=1)

    for l, w in enumerate(layers):
        a = norm(x, w["norm1"])
        bias = {n: w[n].to(f64) if n in w else 0.0 for n in ("bq", "bk", "bv")}
        q = rope((w["wq"].to(f64) @ a + bias["bq"]).view(nq, hd))
        k = rope((w["wk"].to(f64) @ a + bias["bk"]).view(nkv, hd))
        v = (w["wv"].to(f64) @ a + bias["bv"]).view(nkv, hd)
        cache_bf16[l, 0, 0, :, p, :] = k.to(torch.float32).to(torch.bfloat16)
        cache_bf16[l, 1, 0, :, p, :] = v.to(torch.float32).to(torch.bfloat16)
        K = cache_bf16[l, 0, 0, :, : p + 1, :].to(f64).repeat_interleave(nq // nkv, dim=0)  # [nq, n, hd]
        V = cache_bf16[l, 1, 0, :, : p + 1, :].to(f64).repeat_interleave(nq // nkv, dim=0)
        o = F.scaled_dot_product_attention(q.view(1, nq, 1, hd), K.unsqueeze(0), V.unsqueeze(0)).reshape(nq * hd)
        x = x + w["wo"].to(f64) @ o
        m = norm(x, w["norm2"])
        if "router" in w:   # mixture of experts: top-k of the router logits, softmax over the chosen, weighted expert MLPs
            r = w["router"].to(f64) @ m
            val, idx = torch.topk(r, shape.top_k)
            gates = torch.softmax(val, dim=0)
            y = torch.zeros_like(x)
            for g, e in zip(gates, idx.tolist()):
                y = y + g * (w[f"wdown_e{e}"].to(f64) @ (F.silu(w[f"wgate_e{e}"].to(f64) @ m) * (w[f"wup_e{e}"].to(f64) @ m)))
            x = x + y
        else:
            x = x + w["wdown"].to(f64) @ (F.silu(w["wgate"].to(f64) @ m) * (w["wup"].to(f64) @ m))
    logits = glob["lm_head"].to(f64) @ norm(x, glob["norm_f"])
    return x.numpy(), logits.numpy()


def test_whole_step_against_torch_library_restatement_16_greedy_steps():
    shape, layers, glob, cache = _tiny_setup()
    orc = ko.Oracle(shape, cache.shape[4], lambda l: layers[l], glob)
    c_or = u16(cache).copy()
    c_t = cache.clone()
    tok = int(gen.make_tokens(shape, 1, 0)[0])
    p = 128
    for step in range(16):
        hidden, logits, nxt = orc.step(c_or, [tok], [p])
        h_ref, l_ref = _torch_reference_step(shape, layers, glob, c_t, tok, p)
        assert np.allclose(hidden[0], h_ref, rtol=1e-9, atol=1e-11), step
        assert np.allclose(logits[0], l_ref, rtol=1e-9, atol=1e-11), step
        assert int(nxt[0]) == int(np.argmax(l_ref))
        # appended rows agree with torch's own bf16 rounding (a rare double-rounding tie may differ by one ulp)
        same = (c_or[:, :, :, :, p, :] == u16(c_t)[:, :, :, :, p, :]).mean()
        assert same > 0.999
        c_t[:, :, :, :, p, :] = torch.from_numpy(c_or[:, :, :, :, p, :].copy()).view(torch.bfloat16)
        tok, p = int(nxt[0]), p + 1


def test_identity_projections_closed_form():
    """One layer, hidden = q_dim, W_q = W_k = W_v = W_o = I, no cached context (p = 0), W_gate = 0:
    attention over the single new position returns bf16(v) = bf16(a), so x_out = x + bf16(rmsnorm(x))."""
    shape = gen.ModelShape(1, 16, 2, 2, 8, 8, 32, 1e-5, 10000.0)
    eye = torch.eye(16).to(torch.bfloat16)
    lw = gen.make_layer(shape, 0, 11)
    lw = {k: v.clone() for k, v in lw.items()}
    for n in ("wq", "wk", "wv", "wo"):
        lw[n] = eye.clone()
    lw["wgate"].zero_()
    glob = gen.make_globals(shape, 11)
    orc = ko.Oracle(shape, 4, lambda l: lw, glob)
    cache = np.zeros(gen.kv_cache_shape(shape, 1, 4), dtype=np.uint16)
    tok = 9
    x0 = orc.embed(tok)
    hidden, _, _ = orc.step(cache, [tok], [0], want_logits=False)
    a = ko.rmsnorm(x0, u16(lw["norm1"]), shape.rms_eps)
    expect = x0 + ko.bf16_to_double(bf16_of(a.astype(np.float32)))
    # a -> float32 -> bf16 may double-round on a tie; allow one bf16 ulp on that term
    assert np.allclose(hidden[0], expect, rtol=0, atol=2.0 ** -8 * np.abs(a).max())
    assert np.array_equal(ko.bf16_to_double(cache[0, 1, 0, :, 0, :]).reshape(-1), hidden[0] - x0)


# ------------------------------------------------------------------ the paper's printed figures

def _table1():
    rows = []
    with open(GOLDEN / "table1_op_intensity.csv") as f:
        for r in csv.DictReader(line for line in f if not line.startswith("#")):
            rows.append(r)
    return rows


def test_operation_intensity_table():
    """The oracle's own MAC and byte counters, run in count-only mode at the table's shapes, must give the
    printed KV sizes exactly, the printed GFLOPs under the table's rounding, and the printed bytes and
    intensities within the slack of the table's nominal parameter counts."""
    rows = _table1()
    assert len(rows) == 12
    printed_b1 = {(r["model"], int(r["context"])): float(r["gflops"]) for r in rows if r["batch"] == "1"}
    for r in rows:
        shape = SHAPES[r["model"]]
        B, T = int(r["batch"]), int(r["context"])
        c = ko.count_step(shape, B, T - 1)  # the step that brings the context to T positions
        s = shape
        # closed forms of the counters (exact integers)
        matmul_params = s.n_layers * (s.hidden * s.head_dim * (2 * s.n_q_heads + 2 * s.n_kv_heads) + 3 * s.hidden * s.ffn) \
            + s.vocab * s.hidden
        assert c["macs"] == B * (matmul_params + 2 * T * s.n_q_heads * s.head_dim * s.n_layers)
        assert c["kv_read_bytes"] == B * T * s.n_layers * 2 * s.n_kv_heads * s.head_dim * 2
        assert c["weight_bytes"] == 2 * (matmul_params + s.n_layers * 2 * s.hidden + s.hidden)
        assert c["kv_write_bytes"] == B * s.n_layers * 2 * s.n_kv_heads * s.head_dim * 2
        assert c["embed_bytes"] == B * s.hidden * 2
        # KV column (GB = 2^30 bytes; the 405B rows are printed truncated and x32 of the truncated value)
        kv_gb = c["kv_read_bytes"] / 2 ** 30
        printed_kv = float(r["kv_gb"])
        if r["model"] == "405B":
            assert abs(kv_gb - printed_kv) / printed_kv < 0.006
        else:
            assert kv_gb == printed_kv
        # GFLOPs column: batch-1 rows are printed to the nearest ten; batch-32 rows are 32 x the printed batch-1 row
        gflop_b1 = 2 * (c["macs"] // B) / 1e9
        assert abs(gflop_b1 - printed_b1[(r["model"], T)]) <= 10.0
        assert float(r["gflops"]) == B * printed_b1[(r["model"], T)]
        # bytes column = all parameters (embedding table included) + KV, parameters at the nominal model size
        all_param_bytes = c["weight_bytes"] + 2 * s.vocab * s.hidden
        gbytes = (all_param_bytes + c["kv_read_bytes"]) / 2 ** 30
        assert abs(all_param_bytes / 2 ** 30 - float(r["params_gb"])) / float(r["params_gb"]) < 0.01
        assert abs(gbytes - float(r["gbytes"])) / float(r["gbytes"]) < 0.01
        assert abs(float(r["params_gb"]) + printed_kv - float(r["gbytes"])) < 0.11
        # intensity column = printed GFLOPs / printed GBytes; every row is memory-bound on DGX H100 (< 1000/3)
        assert abs(float(r["gflops"]) / float(r["gbytes"]) - float(r["flops_per_byte"])) < 0.06
        assert 2 * c["macs"] / (all_param_bytes + c["kv_read_bytes"]) < 1000.0 / 3.0


def test_counters_match_executed_work():
    """The counters advance identically whether the loops run or are skipped."""
    shape, layers, glob, cache = _tiny_setup()
    orc = ko.Oracle(shape, cache.shape[4], lambda l: layers[l], glob)
    orc.step(u16(cache).copy(), [3], [128])
    assert orc.counters.as_dict() == ko.count_step(shape, 1, 128, cache.shape[4])


def test_kernel_call_counts():
    vals = dict(line.strip().split("=") for line in open(GOLDEN / "call_counts.txt") if "=" in line and not line.startswith("#"))
    L = gen.LLAMA31_8B.n_layers
    assert int(vals["per_operator_launches"]) == L * 10 + 3
    assert int(vals["per_layer_launches"]) == L + 3
    assert int(vals["looped_launches"]) == 1 + 3


# ------------------------------------------------------------------ input generator (shared, arithmetic-free)

def test_generator_statistics_and_determinism():
    t = gen.make_tensor(gen.TINY, "wgate", 2, 0).to(torch.float64)
    assert abs(t.mean().item()) < 3e-4 and abs(t.std().item() - 0.02) < 4e-4
    g = gen.make_tensor(gen.TINY, "norm1", 0, 0).to(torch.float64)
    assert abs(g.mean().item() - 1.0) < 5e-3
    assert torch.equal(gen.make_tensor(gen.TINY, "wq", 1, 0), gen.make_tensor(gen.TINY, "wq", 1, 0))
    assert not torch.equal(gen.make_tensor(gen.TINY, "wq", 1, 0), gen.make_tensor(gen.TINY, "wq", 2, 0))
    assert not torch.equal(gen.make_tensor(gen.TINY, "wq", 1, 0), gen.make_tensor(gen.TINY, "wq", 1, 1))
    kv = gen.make_kv_cache(gen.TINY, 2, 128, 160, 0)
    assert kv.shape == (4, 2, 2, 2, 160, 64)
    assert not kv[:, :, :, :, 128:].any()
    assert abs(kv[:, :, :, :, :128].to(torch.float64).std().item() - 1.0) < 0.01
    toks = gen.make_tokens(gen.TINY, 64, 0)
    assert toks.min() >= 0 and toks.max() < 1024 and toks.unique().numel() > 40
    # embed_rows regenerates table rows without the table
    E = gen.make_tensor(gen.TINY, "embed", -1, 0)
    assert torch.equal(gen.embed_rows(gen.TINY, [5, 1000], 0), E[[5, 1000]])


# ------------------------------------------------------------------ mixture-of-experts layers

def test_moe_router_top_k_order_ties_and_weights():
    """Router of a mixture-of-experts layer: the k largest logits in descending order, the lower index first among
    equals; the weights are the softmax over the chosen logits, which is the softmax over ALL experts restricted to
    the chosen ones and renormalised; k = E is the plain softmax; equal logits give equal weights 1/k."""
    idx, w = ko.moe_route(np.array([0.1, 2.0, 2.0, -1.0, 0.5]), 3)
    assert idx == [1, 2, 4]                                   # tie between experts 1 and 2: the lower index first
    assert abs(w.sum() - 1.0) < 1e-15 and w[0] == w[1] > w[2]
    idx, w = ko.moe_route(np.array([3.0, 3.0, 3.0, 3.0]), 2)
    assert idx == [0, 1] and np.allclose(w, [0.5, 0.5], rtol=0, atol=1e-16)
    idx, w = ko.moe_route(np.array([-5.0, 7.0, 1.0]), 1)
    assert idx == [1] and w[0] == 1.0
    rng = np.random.default_rng(1)
    for _ in range(50):
        E, k = int(rng.integers(2, 17)), 0
        k = int(rng.integers(1, E + 1))
        r = rng.normal(size=E) * 3.0
        idx, w = ko.moe_route(r, k)
        order = sorted(range(E), key=lambda e: (-r[e], e))[:k]          # brute force: sort by (-logit, index)
        assert idx == order
        full = np.exp(r - r.max())
        full /= full.sum()                                              # softmax over all experts ...
        assert np.allclose(w, full[order] / full[order].sum(), rtol=1e-13, atol=0)   # ... restricted and renormalised
        if k == E:
            assert np.allclose(w, full[order], rtol=1e-13, atol=0)


def _moe_shape(**kw):
    return dataclasses.replace(gen.TINY, n_experts=4, top_k=2, **kw)


def test_moe_identical_experts_equal_the_dense_layer():
    """Every expert holds the dense model's MLP matrices: whatever the router picks, the gates sum to one, so the
    mixture-of-experts model computes exactly what the dense model does -- also with k = E and a zero router (all gates
    equal: the plain mean of the experts), and with k = 1 (one expert, gate 1)."""
    dense_shape, dense_layers, glob, cache = _tiny_setup()
    for E, k, zero_router in ((4, 2, False), (4, 4, True), (3, 1, False)):
        shape = dataclasses.replace(dense_shape, n_experts=E, top_k=k)
        layers = []
        for l, lw in enumerate(dense_layers):
            d = {n: t for n, t in lw.items() if n not in ("wgate", "wup", "wdown")}
            d["router"] = gen.make_tensor(shape, "router", l, 0, "cpu")
            if zero_router:
                d["router"] = torch.zeros_like(d["router"])
            for e in range(E):
                d[f"wgate_e{e}"], d[f"wup_e{e}"], d[f"wdown_e{e}"] = lw["wgate"], lw["wup"], lw["wdown"]
            layers.append(d)
        c_moe, c_dense = u16(cache).copy(), u16(cache).copy()
        moe = ko.Oracle(shape, cache.shape[4], lambda l: layers[l], glob)
        dense = ko.Oracle(dense_shape, cache.shape[4], lambda l: dense_layers[l], glob)
        h1, l1, n1 = moe.step(c_moe, [5], [128])
        h2, l2, n2 = dense.step(c_dense, [5], [128])
        assert np.allclose(h1, h2, rtol=1e-12, atol=1e-13) and np.allclose(l1, l2, rtol=1e-11, atol=1e-12)
        assert n1[0] == n2[0] and np.array_equal(c_moe, c_dense)


def test_moe_whole_step_against_torch_library_restatement():
    """Mixture-of-experts decoder (4 experts, 2 per token, all different) against the torch re-statement (topk,
    softmax, matmul) for 8 greedy steps."""
    shape = _moe_shape()
    layers = [gen.make_layer(shape, l, 3, "cpu") for l in range(shape.n_layers)]
    glob = gen.make_globals(shape, 3, "cpu")
    cache = gen.make_kv_cache(shape, 1, 64, 80, 3, "cpu")
    orc = ko.Oracle(shape, 80, lambda l: layers[l], glob)
    c_or, c_ref = u16(cache).copy(), cache.clone()
    tok = 11
    for step in range(8):
        p = 64 + step
        hidden, logits, nxt = orc.step(c_or, [tok], [p])
        h_ref, l_ref = _torch_reference_step(shape, layers, glob, c_ref, tok, p)
        assert np.allclose(hidden[0], h_ref, rtol=1e-10, atol=1e-11)
        assert np.allclose(logits[0], l_ref, rtol=1e-9, atol=1e-10)
        assert np.array_equal(c_or, u16(c_ref))
        assert int(nxt[0]) == int(np.argmax(l_ref))
        tok = int(nxt[0])
    # the counters: a mixture-of-experts layer touches the router and top_k experts, not all of them
    cnt = ko.count_step(shape, 1, 64)
    per_expert = 3 * shape.hidden * shape.ffn
    attn = shape.hidden * shape.head_dim * (2 * shape.n_q_heads + 2 * shape.n_kv_heads)
    mlp = shape.top_k * per_expert + shape.n_experts * shape.hidden
    assert cnt["weight_bytes"] == 2 * (shape.n_layers * (attn + mlp + 2 * shape.hidden) + shape.hidden + shape.vocab * shape.hidden)
