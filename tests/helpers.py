"""Shared test plumbing: builds the same seeded model for the CUDA path and for the oracle, runs teacher-forced
decode on both and compares.  No arithmetic of the method lives here."""
from __future__ import annotations

import numpy as np
import torch

from oracle import kl_oracle as ko
from paper_2410_23668_b200 import binding, build, inputs as gen

# spec tolerances (bf16 weights / KV, fp32 accumulation on the GPU, fp64 oracle)
REL_L2_TOL = 1e-2
ABS_LOGIT_TOL = 5e-2


def gen_device():
    return "cuda" if torch.cuda.is_available() else "cpu"


class HostWeights:
    """Weights for the oracle: generated (on the GPU when there is one, bit-identical either way) and kept on the
    host, or regenerated layer by layer when `stream_layers` is set."""

    def __init__(self, shape, seed, stream_layers=False, overrides=None):
        self.shape, self.seed, self.stream = shape, seed, stream_layers
        self.overrides = overrides or {}
        self._cache = {}

    def _apply(self, l, d):
        for (name, layer), t in self.overrides.items():
            if layer == l and name in d:
                d[name] = t.cpu()
        return d

    def layer(self, l):
        if l in self._cache:
            return self._cache[l]
        d = {k: v.cpu() for k, v in gen.make_layer(self.shape, l, self.seed, gen_device()).items()}
        d = self._apply(l, d)
        if not self.stream:
            self._cache[l] = d
        return d

    def globals(self, with_table=True):
        if "g" not in self._cache:
            g = {k: v.cpu() for k, v in gen.make_globals(self.shape, self.seed, gen_device(), with_table).items()}
            if not with_table:
                g["embed_row"] = lambda tok: gen.embed_rows(self.shape, [tok], self.seed)[0]
            self._cache["g"] = self._apply(-1, g)
        return self._cache["g"]


def make_decoder(shape, max_batch, max_ctx, seed, overrides=None, stash=True):
    """CUDA-path model with weights generated on the device, one layer at a time.  stash=False keeps the batch-1
    kernels in their plain mode on shapes that would take the stash mode."""
    build.build_library()
    dec = binding.Decoder(shape, max_batch, max_ctx, stash=stash)
    overrides = overrides or {}
    for l in range(shape.n_layers):
        for name, t in gen.make_layer(shape, l, seed, "cuda").items():
            t = overrides.get((name, l), t)
            dec.kl_load_weights(name, l, t.cuda())
        torch.cuda.synchronize()
    for name, t in gen.make_globals(shape, seed, "cuda").items():
        t = overrides.get((name, -1), t)
        dec.kl_load_weights(name, -1, t.cuda())
    torch.cuda.synchronize()
    return dec


def rel_l2(a: np.ndarray, ref: np.ndarray) -> float:
    return float(np.linalg.norm(a.astype(np.float64) - ref) / max(np.linalg.norm(ref), 1e-30))


def bf16_decode(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def run_parity(shape, context, steps, seed=0, batch=1, max_ctx=None,
               modes=(binding.KL_MODE_LOOPED, binding.KL_MODE_PER_LAYER, binding.KL_MODE_PER_STAGE),
               overrides=None, positions0=None, stream_layers=False, check_cache=True, batched_path=None, stash=True):
    """Teacher-forced greedy decode: the oracle runs `steps` steps on its own tokens; each CUDA mode consumes the
    oracle's token of the previous step.  Returns a report dict; asserts nothing.  batched_path: None leaves the
    library's default (batches take the tensor-core path when the shape allows), True / False forces the choice
    (True raises when the shape has no such path)."""
    max_ctx = max_ctx or (context + steps + 8)
    host = HostWeights(shape, seed, stream_layers, overrides)
    orc = ko.Oracle(shape, max_ctx, host.layer, host.globals())
    cache0 = gen.make_kv_cache(shape, batch, context, max_ctx, seed, gen_device())
    cache_or = cache0.cpu().view(torch.uint16).numpy().copy()
    toks = gen.make_tokens(shape, batch, seed).tolist()
    pos = list(positions0) if positions0 is not None else [context] * batch

    ref = []
    t, p = list(toks), list(pos)
    for s in range(steps):
        hidden, logits, nxt = orc.step(cache_or, t, p)
        srt = np.sort(logits, axis=1)
        ref.append(dict(tokens=list(t), positions=list(p), hidden=hidden, logits=logits, next=nxt.tolist(),
                        margin=(srt[:, -1] - srt[:, -2]).tolist()))
        t, p = nxt.tolist(), [q + 1 for q in p]

    report = dict(ref=ref, modes={}, cache_ref=cache_or, cache0=cache0.cpu().view(torch.uint16).numpy())
    dec = make_decoder(shape, batch, max_ctx, seed, overrides, stash)
    report["stash_mode"] = dec.kl_stash_mode()
    if batched_path is not None:
        dec.kl_set_batched_path(batched_path)
    for mode in modes:
        dec.kl_set_mode(mode)
        cache = cache0.clone().cuda()
        logits_d = torch.empty(batch, shape.vocab, dtype=torch.float32, device="cuda")
        hidden_d = torch.empty(batch, shape.hidden, dtype=torch.float32, device="cuda")
        rows = []
        for s in range(steps):
            tok_d = torch.tensor(ref[s]["tokens"], dtype=torch.int32, device="cuda")
            pos_d = torch.tensor(ref[s]["positions"], dtype=torch.int32, device="cuda")
            dec.kl_decode_step(tok_d, pos_d, cache, logits_d, batch)
            dec.kl_read_hidden(hidden_d, batch)
            dec.kl_argmax_advance(logits_d, tok_d, pos_d, batch)
            torch.cuda.synchronize()
            st = dec.kl_last_status()
            lg, hd = logits_d.cpu().numpy(), hidden_d.cpu().numpy()
            rows.append(dict(status=st, logits=lg, hidden=hd, next=tok_d.cpu().tolist(), pos_after=pos_d.cpu().tolist(),
                             rel_hidden=max(rel_l2(hd[b], ref[s]["hidden"][b]) for b in range(batch)),
                             rel_logits=max(rel_l2(lg[b], ref[s]["logits"][b]) for b in range(batch)),
                             max_abs_logit=float(np.abs(lg - ref[s]["logits"]).max())))
        report["modes"][mode] = dict(steps=rows, cache=cache.cpu().view(torch.uint16).numpy() if check_cache else None)
    dec.close()
    return report


def assert_parity(report, steps, batch=1, check_cache=True, flip_tol=0.02):
    ref = report["ref"]
    for mode, res in report["modes"].items():
        for s in range(steps):
            r = res["steps"][s]
            assert r["status"] == 0, (mode, s, r["status"])
            assert np.isfinite(r["logits"]).all(), (mode, s)
            assert r["rel_hidden"] <= REL_L2_TOL, (mode, s, r["rel_hidden"])
            assert r["rel_logits"] <= REL_L2_TOL, (mode, s, r["rel_logits"])
            assert r["max_abs_logit"] <= ABS_LOGIT_TOL, (mode, s, r["max_abs_logit"])
            assert r["next"] == ref[s]["next"], (mode, s, r["next"], ref[s]["next"], ref[s]["margin"])
            assert r["pos_after"] == [q + 1 for q in ref[s]["positions"]]
        if check_cache and res["cache"] is not None:
            # prefilled rows are untouched (bit-exact); rows appended by the steps hold bf16 roundings of values
            # computed in fp32 here and fp64 in the oracle: equal up to one bf16 rounding step of a ~1e-5 difference
            got, exp = res["cache"], report["cache_ref"]
            changed = (exp != report["cache0"])
            assert np.array_equal(got[~changed], exp[~changed]), mode
            g, e = bf16_decode(got[changed]), bf16_decode(exp[changed])
            assert np.all(np.abs(g - e) <= 2.0 ** -7 * np.abs(e) + 1e-3 * np.abs(e).max()), mode
            assert (got[changed] != exp[changed]).mean() < flip_tol, mode
    modes = list(report["modes"].values())
    for other in modes[1:]:  # the transformation preserves semantics: all schedules run the same arithmetic
        for s in range(steps):
            assert np.array_equal(modes[0]["steps"][s]["logits"], other["steps"][s]["logits"]), s
            assert np.array_equal(modes[0]["steps"][s]["hidden"], other["steps"][s]["hidden"]), s
        if modes[0]["cache"] is not None:
            assert np.array_equal(modes[0]["cache"], other["cache"])


def run_full_depth(shape, context, steps, batch=1, oracle_rows=None, seed=0, batched_path=None, greedy_chain=False):
    """Teacher-forced decode through ALL layers of a large model, compared with the layer-streaming oracle.

    The oracle decodes the sequences `oracle_rows` (default: all) of the batch -- sequences are independent, so a subset
    is exact; the CUDA path decodes the whole batch.  Sequences the oracle does not run continue on the tokens the
    CUDA path picked itself and are checked for finite logits only.  The cache is compared on the rows appended by the
    steps (the prefilled rows of a multi-gigabyte cache are not copied back).  greedy_chain: the CUDA path decodes
    through kl_decode_greedy (one launch per token at batch 1), not kl_decode_step + kl_argmax_advance.
    Asserts the benchmark spec's tolerances; returns the worst errors seen."""
    rows = list(range(batch)) if oracle_rows is None else list(oracle_rows)
    max_ctx = context + steps + 8
    host = HostWeights(shape, seed, stream_layers=True)
    orc = ko.Oracle(shape, max_ctx, host.layer, host.globals(with_table=False))
    cache = gen.make_kv_cache(shape, batch, context, max_ctx, seed, "cuda")
    cache_or = cache[:, :, rows].cpu().view(torch.uint16).numpy().copy()
    toks = gen.make_tokens(shape, batch, seed).tolist()
    ref = []
    t, p = [toks[r] for r in rows], [context] * len(rows)
    for s in range(steps):
        hidden, logits, nxt = orc.step(cache_or, t, p)
        srt = np.sort(logits, axis=1)
        ref.append(dict(tokens=list(t), hidden=hidden, logits=logits, next=nxt.tolist(), margin=(srt[:, -1] - srt[:, -2]).tolist()))
        t, p = nxt.tolist(), [q + 1 for q in p]
    dec = make_decoder(shape, batch, max_ctx, seed)
    if batched_path is not None:
        dec.kl_set_batched_path(batched_path)
    tok_d = torch.tensor(toks, dtype=torch.int32, device="cuda")
    pos_d = torch.full((batch,), context, dtype=torch.int32, device="cuda")
    logits_d = torch.empty(batch, shape.vocab, dtype=torch.float32, device="cuda")
    hidden_d = torch.empty(batch, shape.hidden, dtype=torch.float32, device="cuda")
    worst = dict(rel_hidden=0.0, rel_logits=0.0, max_abs_logit=0.0)
    for s in range(steps):
        tok_d[rows] = torch.tensor(ref[s]["tokens"], dtype=torch.int32, device="cuda")   # teacher forcing
        if greedy_chain:
            dec.kl_decode_greedy(tok_d, pos_d, cache, logits_d, batch, True)
        else:
            dec.kl_decode_step(tok_d, pos_d, cache, logits_d, batch)
            dec.kl_argmax_advance(logits_d, tok_d, pos_d, batch)
        dec.kl_read_hidden(hidden_d, batch)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == 0, s
        lg, hd = logits_d.cpu().numpy(), hidden_d.cpu().numpy()
        assert np.isfinite(lg).all() and np.isfinite(hd).all(), s
        assert pos_d.cpu().tolist() == [context + s + 1] * batch
        nxt = tok_d.cpu().tolist()
        for i, r in enumerate(rows):
            e = dict(rel_hidden=rel_l2(hd[r], ref[s]["hidden"][i]), rel_logits=rel_l2(lg[r], ref[s]["logits"][i]),
                     max_abs_logit=float(np.abs(lg[r] - ref[s]["logits"][i]).max()))
            assert e["rel_hidden"] <= REL_L2_TOL and e["rel_logits"] <= REL_L2_TOL and e["max_abs_logit"] <= ABS_LOGIT_TOL, (s, r, e)
            assert nxt[r] == ref[s]["next"][i], (s, r, nxt[r], ref[s]["next"][i], ref[s]["margin"][i])
            for k in worst:
                worst[k] = max(worst[k], e[k])
    # rows appended by the steps: within one bf16 rounding step of the oracle's (fp32 here, fp64 there)
    got = cache[:, :, rows, :, context:context + steps].cpu().view(torch.uint16).numpy()
    exp = cache_or[:, :, :, :, context:context + steps]
    g, e = bf16_decode(got), bf16_decode(exp)
    assert np.all(np.abs(g - e) <= 2.0 ** -7 * np.abs(e) + 1e-3 * np.abs(e).max())
    worst["cache_values_differing"] = float((got != exp).mean())
    dec.close()
    return worst
