#!/usr/bin/env python
"""Decode-throughput benchmark of the kernel-looped decoder (one JSON line on stdout).

A step is one pass of the whole hot path -- Embedding, L decoder layers, Classifier, greedy Sampling -- for one
batch of sequences.  Default workload: Llama-3.1-8B shape, batch 1, context 4096 (the configuration the paper's
operation-intensity table and headline figure are quoted on), synthetic seeded weights and KV cache.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

N > 1 (under torchrun) runs N independent replicas: a decode stream is a strict chain, so the path does not shard
and no data-path collective exists; torch.distributed is used for the barrier and the max-over-ranks only.
`--impl reference` times the CPU oracle on the host cores, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import torch

from paper_2410_23668_b200 import inputs as gen

WORKLOADS = {
    # name: (shape, batch, context, default steps)
    "tiny_b1_ctx128": (gen.TINY, 1, 128, 16),
    "llama31_8b_b1_ctx4096": (gen.LLAMA31_8B, 1, 4096, 128),
    # four layers of the same shape: a few GB on the device, for multi-pass profiler captures
    "llama31_8b_4layers_b1_ctx4096": (gen.ModelShape(4, 4096, 32, 8, 128, 14336, 128256, 1e-5, 500000.0), 1, 4096, 8),
    "llama31_8b_b1_ctx65536": (gen.LLAMA31_8B, 1, 65536, 64),
    "llama31_70b_b1_ctx4096": (gen.LLAMA31_70B, 1, 4096, 32),
    # batches take the tensor-core path: every projection one dense contraction for the whole batch
    "llama31_8b_b32_ctx4096": (gen.LLAMA31_8B, 32, 4096, 16),
    # batch sizes and context lengths of the paper's Table 2 (8 and 16 sequences, 8K and 16K tokens), same decoder shape
    "llama31_8b_b2_ctx4096": (gen.LLAMA31_8B, 2, 4096, 32),
    "llama31_8b_b4_ctx4096": (gen.LLAMA31_8B, 4, 4096, 32),
    "llama31_8b_b8_ctx4096": (gen.LLAMA31_8B, 8, 4096, 32),
    "llama31_8b_b16_ctx4096": (gen.LLAMA31_8B, 16, 4096, 16),
    "llama31_8b_b8_ctx8192": (gen.LLAMA31_8B, 8, 8192, 16),
    "llama31_8b_b16_ctx16384": (gen.LLAMA31_8B, 16, 16384, 16),
    "llama31_70b_b8_ctx4096": (gen.LLAMA31_70B, 8, 4096, 8),
    # the 72B decoder of Table 2 by its public dimensions (biases on the q, k, v projections)
    "qwen25_72b_shape_b1_ctx4096": (gen.ModelShape(80, 8192, 64, 8, 128, 29568, 152064, 1e-6, 1000000.0, True), 1, 4096, 16),
    "qwen25_72b_shape_b8_ctx4096": (gen.ModelShape(80, 8192, 64, 8, 128, 29568, 152064, 1e-6, 1000000.0, True), 8, 4096, 8),
    # the 3B decoder of Table 2 by its public dimensions
    "llama32_3b_b1_ctx4096": (gen.ModelShape(28, 3072, 24, 8, 128, 8192, 128256, 1e-5, 500000.0), 1, 4096, 64),
    "llama32_3b_b16_ctx8192": (gen.ModelShape(28, 3072, 24, 8, 128, 8192, 128256, 1e-5, 500000.0), 16, 8192, 16),
    # the mixture-of-experts decoder of Table 2 by its public dimensions: 8 experts of FFN 14336, 2 per token (93 GB of
    # weights, of which a step reads 25 GB)
    "mixtral_8x7b_shape_b1_ctx4096": (gen.ModelShape(32, 4096, 32, 8, 128, 14336, 32000, 1e-5, 1000000.0, False, 8, 2), 1, 4096, 32),
    "llama31_70b_2layers_b8_ctx4096": (gen.ModelShape(2, 8192, 64, 8, 128, 28672, 128256, 1e-5, 500000.0), 8, 4096, 4),
    # two layers, 32 sequences at the full context: a few GB on the device, for profiler captures of the batched path
    "llama31_8b_2layers_b32_ctx4096": (gen.ModelShape(2, 4096, 32, 8, 128, 14336, 128256, 1e-5, 500000.0), 32, 4096, 4),
}
DEFAULT_WORKLOAD = "llama31_8b_b1_ctx4096"
NOMINAL_HBM_GBS = 8000.0


def layer_weight_bytes(s) -> int:
    """Weight bytes one decode step reads per layer.  A mixture-of-experts layer reads its router and the top_k chosen
    experts, not all of them."""
    mlp = 3 * s.hidden * s.ffn
    if getattr(s, "n_experts", 0):
        mlp = s.top_k * mlp + s.n_experts * s.hidden
    return 2 * (s.hidden * s.head_dim * (2 * s.n_q_heads + 2 * s.n_kv_heads) + mlp + 2 * s.hidden)


def kv_bytes(s, batch: int, position: int) -> int:
    """KV rows 0..position-1 read plus row `position` written, every layer."""
    return batch * s.n_layers * 2 * s.n_kv_heads * s.head_dim * 2 * (position + 1)


def decoder_bytes(s, batch: int, position: int) -> int:
    """Algorithmic HBM bytes of the decoder kernel(s) of one step: all layers' matrices and gains once + KV."""
    return s.n_layers * layer_weight_bytes(s) + kv_bytes(s, batch, position)


def step_bytes(s, batch: int, position: int) -> int:
    """Algorithmic HBM bytes of one whole step: decoder + final gain + lm_head + B embedding rows."""
    return decoder_bytes(s, batch, position) + 2 * s.hidden + 2 * s.vocab * s.hidden + batch * 2 * s.hidden


def measured_peaks() -> dict:
    f = ROOT / "MEASURED_PEAKS.json"
    if f.exists():
        d = json.loads(f.read_text())
        return {"hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) while the timed regions run."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            visible = os.environ.get("CUDA_VISIBLE_DEVICES")
            phys = index
            if visible:
                ids = [v for v in visible.split(",") if v.strip() != ""]
                if index < len(ids) and ids[index].strip().isdigit():
                    phys = int(ids[index])
            self.h = pynvml.nvmlDeviceGetHandleByIndex(phys)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


def build_model(shape, batch, context, steps_total, seed=0, stash=True):
    from paper_2410_23668_b200 import binding
    max_ctx = context + steps_total + 8
    dec = binding.Decoder(shape, batch, max_ctx, stash=stash)
    for l in range(shape.n_layers):
        for name, t in gen.make_layer(shape, l, seed, "cuda").items():
            dec.kl_load_weights(name, l, t)
        torch.cuda.synchronize()
    for name, t in gen.make_globals(shape, seed, "cuda").items():
        dec.kl_load_weights(name, -1, t)
    torch.cuda.synchronize()
    cache = gen.make_kv_cache(shape, batch, context, max_ctx, seed, "cuda")
    return dec, cache, max_ctx


def run_device_loop(dec, cache, tok0, context, batch, warmup, steps, stream):
    """W + K greedy steps with tokens and positions resident on the device; returns ms for the K timed steps."""
    tok = tok0.clone()
    pos = torch.full((batch,), context, dtype=torch.int32, device="cuda")
    logits = torch.empty(batch, dec.shape.vocab, dtype=torch.float32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for _ in range(warmup):
        dec.kl_decode_step(tok, pos, cache, logits, batch, stream)
        dec.kl_argmax_advance(logits, tok, pos, batch, stream)
    torch.cuda.synchronize()
    barrier()
    e0.record(stream)
    for _ in range(steps):
        dec.kl_decode_step(tok, pos, cache, logits, batch, stream)
        dec.kl_argmax_advance(logits, tok, pos, batch, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    st = dec.kl_last_status()
    if st != 0:
        raise RuntimeError(f"device status {st} after the timed loop")
    return e0.elapsed_time(e1)


def run_token_loop(dec, cache, tok0, context, batch, warmup, steps, stream):
    """Greedy decoding with kl_decode_greedy chained on the device: at batch 1 one launch per token (decoder layers,
    classifier and sampling in one persistent kernel that also prepares the next token's embedding)."""
    tok = tok0.clone()
    pos = torch.full((batch,), context, dtype=torch.int32, device="cuda")
    logits = torch.empty(batch, dec.shape.vocab, dtype=torch.float32, device="cuda")
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(warmup):
        dec.kl_decode_greedy(tok, pos, cache, logits, batch, i == 0, stream)
    torch.cuda.synchronize()
    barrier()
    e0.record(stream)
    for _ in range(steps):
        dec.kl_decode_greedy(tok, pos, cache, logits, batch, False, stream)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    st = dec.kl_last_status()
    if st != 0:
        raise RuntimeError(f"device status {st} after the chained steps")
    assert int(pos[0]) == context + warmup + steps
    return e0.elapsed_time(e1)


def run_tokens_per_launch(dec, cache, tok0, context, warmup, steps, stream, host=False):
    """Batch 1: the K timed steps as ONE call of kl_decode_greedy_tokens (the loop over layers extended to a loop over
    tokens: up to 256 tokens per launch) behind `warmup` chained one-token launches.  host=True: through the host-buffer
    entry point instead (token and position in, K tokens out, synchronised), timed by the host clock."""
    tok = tok0.clone()
    pos = torch.full((1,), context, dtype=torch.int32, device="cuda")
    logits = torch.empty(1, dec.shape.vocab, dtype=torch.float32, device="cuda")
    out = torch.empty(steps, dtype=torch.int32, device="cuda")
    out_h = torch.empty(steps, dtype=torch.int32).pin_memory()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(warmup):
        dec.kl_decode_greedy(tok, pos, cache, logits, 1, i == 0, stream)
    torch.cuda.synchronize()
    barrier()
    if host:
        t0 = time.perf_counter()
        done, token, position = 0, int(tok[0]), context + warmup
        while done < steps:
            n = min(256, steps - done)
            dec.kl_decode_greedy_tokens_host(token, position, cache, out_h[done:], n, stream)
            done, token, position = done + n, int(out_h[done + n - 1]), position + n
        ms = (time.perf_counter() - t0) * 1e3
    else:
        e0.record(stream)
        dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out, steps, 1, False, stream)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        assert int(pos[0]) == context + warmup + steps
    barrier()
    st = dec.kl_last_status()
    if st != 0:
        raise RuntimeError(f"device status {st} after kl_decode_greedy_tokens")
    return ms


def run_graph_loop(dec, cache, tok0, context, batch, warmup, steps, greedy=False):
    """The same greedy steps with ONE decode step (all its launches + sampling) captured in a CUDA graph and replayed:
    the launch-overhead-free version of a schedule.  Returns ms for the K timed replays, or None with the reason when
    the capture is refused."""
    tok = tok0.clone()
    pos = torch.full((batch,), context, dtype=torch.int32, device="cuda")
    logits = torch.empty(batch, dec.shape.vocab, dtype=torch.float32, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    try:
        def one(first):
            if greedy:   # the chained one-launch step: the graph holds the single kernel
                dec.kl_decode_greedy(tok, pos, cache, logits, batch, first, side)
            else:
                dec.kl_decode_step(tok, pos, cache, logits, batch, side)
                dec.kl_argmax_advance(logits, tok, pos, batch, side)
        with torch.cuda.stream(side):
            one(True)                                                      # set-up outside the capture
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                one(False)
    except Exception as exc:  # capture not possible on this driver: report it, the plain launches stand
        torch.cuda.synchronize()
        return None, f"{type(exc).__name__}: {exc}".splitlines()[0][:200]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(side):
        for _ in range(warmup):
            graph.replay()
        side.synchronize()
        barrier()
        e0.record(side)
        for _ in range(steps):
            graph.replay()
        e1.record(side)
        side.synchronize()
    barrier()
    st = dec.kl_last_status()
    if st != 0:
        return None, f"device status {st} after the replays"
    if int(pos[0]) != context + 1 + warmup + steps:
        return None, f"positions advanced to {int(pos[0])}, expected {context + 1 + warmup + steps}"
    return e0.elapsed_time(e1), None


def run_host_loop(dec, cache, tok0, context, batch, warmup, steps, stream):
    """End to end through the host-buffer entry point: every step copies tokens and positions host->device,
    runs the step, copies the logits device->host, and the host picks the next token."""
    V = dec.shape.vocab
    tok_h = tok0.cpu().pin_memory()
    pos_h = torch.full((batch,), context, dtype=torch.int32).pin_memory()
    logits_h = torch.empty(batch, V, dtype=torch.float32).pin_memory()

    def one():
        dec.kl_decode_step_host(tok_h, pos_h, cache, logits_h, batch, stream)
        tok_h.copy_(logits_h.argmax(dim=1).to(torch.int32))
        pos_h.add_(1)

    for _ in range(warmup):
        one()
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        one()
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    return e0.elapsed_time(e1)


def run_greedy_host_loop(dec, cache, tok0, context, batch, warmup, steps, stream):
    """End to end greedy decoding through kl_decode_greedy_host: every step copies tokens and positions host->device
    from pinned memory, runs the step and the sampling on the device, and reads the next tokens back to the host."""
    tok_h = tok0.cpu().pin_memory()
    pos_h = torch.full((batch,), context, dtype=torch.int32).pin_memory()
    nxt_h = torch.empty(batch, dtype=torch.int32).pin_memory()

    def one():
        dec.kl_decode_greedy_host(tok_h, pos_h, cache, nxt_h, batch, stream)
        tok_h.copy_(nxt_h)
        pos_h.add_(1)

    for _ in range(warmup):
        one()
    torch.cuda.synchronize()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        one()
    e1.record(stream)
    torch.cuda.synchronize()
    barrier()
    return e0.elapsed_time(e1)


_DIST = {"on": False}


def barrier():
    if _DIST["on"]:
        torch.distributed.barrier()


def max_over_ranks(v: float) -> float:
    if not _DIST["on"]:
        return v
    dev = "cuda" if torch.distributed.get_backend() == "nccl" else "cpu"
    t = torch.tensor([v], dtype=torch.float64, device=dev)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return float(t.item())


def replica_throughput(steps: int, batch: int, world: int, ms_local: float) -> tuple[float, float]:
    """Replicas only: every rank decodes steps x batch tokens of its own stream; the job's time is the slowest
    rank's.  Returns (tokens/s of the whole job, that time in ms).  Collective: one all-reduce(max) of a scalar."""
    ms = max_over_ranks(ms_local)
    return steps * batch * world / (ms * 1e-3), ms


def oracle_layers_that_fit(shape, budget_bytes=24e9) -> int:
    """Decoder layers whose weights the oracle's host can hold at once: all of them for models up to the 8B shape (whole
    decode steps are executed), a bounded sample for the larger ones."""
    stored = layer_weight_bytes(shape)
    if getattr(shape, "n_experts", 0):   # the host holds every expert
        stored += 2 * 3 * shape.hidden * shape.ffn * (shape.n_experts - shape.top_k)
    return shape.n_layers if shape.n_layers * stored <= budget_bytes else 0


class OracleSampler:
    """The oracle, as it stands, on one decode step of a workload: `n_layers_sample` decoder layers (weights and cache
    of those layers only) plus the classifier.  With all layers this is the WHOLE step, the hidden state chained
    through every layer; with fewer it is a bounded sample whose layer time is scaled to the full depth.  Inputs are
    generated once; `step()` only times oracle calls and returns seconds per token."""

    def __init__(self, shape, batch, context, n_layers_sample, seed=0, with_classifier=True):
        from oracle import kl_oracle as ko
        import numpy as np
        self.ko, self.np = ko, np
        self.shape, self.batch, self.context, self.n = shape, batch, context, n_layers_sample
        self.with_classifier = with_classifier
        dev = "cuda" if torch.cuda.is_available() else "cpu"   # where the seeded inputs are generated; the oracle is CPU
        max_ctx = context + 8
        layers = {l: {k: v.cpu() for k, v in gen.make_layer(shape, l, seed, dev).items()} for l in range(self.n)}
        self.glob = {k: v.cpu() for k, v in gen.make_globals(shape, seed, dev, with_embed_table=False).items()}
        self.glob["embed_row"] = lambda tok: gen.embed_rows(shape, [tok], seed)[0]
        self.orc = ko.Oracle(shape, max_ctx, lambda l: layers[l], self.glob)
        self.cache = np.zeros(gen.kv_cache_shape(shape, batch, max_ctx), dtype=np.uint16)
        for l in range(self.n):
            blk = torch.zeros(gen.kv_cache_shape(shape, batch, max_ctx)[1:], dtype=torch.bfloat16, device=dev)
            gen.fill_kv_layer(shape, blk, l, context, seed)
            self.cache[l] = blk.cpu().view(torch.uint16).numpy()
        self.toks = gen.make_tokens(shape, batch, seed).tolist()
        self.threads = ko.num_threads()
        self.t_layers = self.t_cls = 0.0

    def step(self) -> float:
        import ctypes as C
        ko, np, shape = self.ko, self.np, self.shape
        t0 = time.perf_counter()
        hidden, _, _ = self.orc.step(self.cache, self.toks, [self.context] * self.batch, layers=range(self.n),
                                     want_logits=False)
        self.t_layers = time.perf_counter() - t0
        self.t_cls = 0.0
        if self.with_classifier:
            logits = np.empty(shape.vocab, dtype=np.float64)
            t0 = time.perf_counter()
            for b in range(self.batch):
                ko.lib().ko_classifier(C.byref(self.orc.desc), C.c_void_p(ko.as_u16(self.glob["norm_f"]).ctypes.data),
                                       C.c_void_p(ko.as_u16(self.glob["lm_head"]).ctypes.data),
                                       hidden[b].ctypes.data_as(C.POINTER(C.c_double)),
                                       logits.ctypes.data_as(C.POINTER(C.c_double)), None, 0)
            self.t_cls = time.perf_counter() - t0
        return (self.t_layers * shape.n_layers / self.n + self.t_cls) / self.batch

    def describe(self) -> str:
        cls = (f" + classifier executed ({self.t_cls:.2f} s)" if self.with_classifier
               else "; classifier time taken from one separate execution")
        if self.n == self.shape.n_layers:
            return (f"one WHOLE decode step at position {self.context}: all {self.n} decoder layers executed "
                    f"({self.t_layers:.2f} s){cls}, nothing scaled")
        return (f"one decode step at position {self.context}: {self.n} of {self.shape.n_layers} decoder layers "
                f"executed ({self.t_layers:.2f} s){cls}, layer time scaled to {self.shape.n_layers} layers")


def oracle_sample(shape, batch, context, n_layers_sample, seed=0, device="cpu"):
    """One timed sample (see OracleSampler).  Returns (seconds per token, description, threads)."""
    smp = OracleSampler(shape, batch, context, n_layers_sample, seed)
    sec = smp.step()
    return sec, smp.describe(), smp.threads


def run_reference(args, shape, batch, context):
    """Reference arm = the CPU oracle on the host cores.  For models whose weights the host holds at once (up to the 8B
    shape) every step is a WHOLE decode step of the workload -- all layers, classifier, the hidden state chained
    through -- executed for as many of the W + K steps as about two minutes allow (the count is reported; steps beyond
    it take the mean of the executed ones).  For larger models a step is a bounded sample: one decoder layer (scaled to
    the full depth) plus the classifier."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import kl_oracle as ko
    ko.build()
    n = oracle_layers_that_fit(shape) or 1
    whole = n == shape.n_layers
    smp = OracleSampler(shape, batch, context, n, with_classifier=True)
    t_start = time.perf_counter()
    sec_first = smp.step()                       # untimed warm-up / calibration (pages the weights in)
    t_one = smp.t_layers + smp.t_cls
    total = args.steps + args.warmup
    afford = max(1, min(total, int(120.0 / max(t_one, 1e-3))))
    times, executed = [], 0
    for i in range(total):
        if i < afford:
            sec = smp.step()
            executed += 1
        else:
            sec = statistics.mean(times) if times else sec_first
        if i >= args.warmup or not times:
            times.append(sec)
    sec = statistics.mean(times)
    value = 1.0 / sec
    what = (f"WHOLE decode steps at position {context} (all {shape.n_layers} layers + classifier, nothing scaled)" if whole else
            f"bounded samples of a decode step at position {context}: {n} of {shape.n_layers} decoder layers executed and "
            f"scaled to {shape.n_layers}, + the classifier")
    desc = (f"{what}; {executed} of the {total} warm-up + timed steps executed ({time.perf_counter() - t_start:.0f} s of oracle "
            f"time), the others take the mean of the executed ones")
    line = {
        "impl": "reference", "metric": "decode tokens/s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3 * batch, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, "batch": batch, "context": context, "l2": "inputs larger than L2 (weights and KV streamed once per step)"},
        "steps_executed": executed, "whole_steps": whole,
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": smp.threads, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def run_ours(args, shape, batch, context):
    from paper_2410_23668_b200 import binding, build
    if build.needs_build():
        build.build_library()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local))
        _DIST["on"] = True
    K, W = args.steps, max(args.warmup, 3)
    passes = 10  # looped, per-layer, per-stage, one launch per token, profiled, two end-to-end passes, graph replays
    dec, cache, max_ctx = build_model(shape, batch, context, passes * (K + W), seed=rank)
    tok0 = gen.make_tokens(shape, batch, rank, device="cuda")
    stream = torch.cuda.current_stream()
    cache0 = cache.clone() if cache.numel() * 2 < (8 << 30) else None

    def fresh_cache():
        if cache0 is not None:
            cache.copy_(cache0)
        return cache

    sampler = ClockSampler(local)
    sampler.start()
    # 1. headline: looped, device-resident
    dec.kl_set_mode(binding.KL_MODE_LOOPED)
    l0 = dec.kl_launch_count()
    ms_looped = max_over_ranks(run_device_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream))
    launches = (dec.kl_launch_count() - l0) * K // (K + W)
    # 2. the synchronisation-boundary schedule: one launch per layer
    dec.kl_set_mode(binding.KL_MODE_PER_LAYER)
    ms_layer = max_over_ranks(run_device_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream))
    # 2a. the schedule with a kernel boundary after every operator group (five launches per layer)
    dec.kl_set_mode(binding.KL_MODE_PER_STAGE)
    ms_stage = max_over_ranks(run_device_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream))
    # 2c. one launch per token: decoder layers, classifier and sampling in one kernel (kl_decode_greedy, chained)
    l0t = dec.kl_launch_count()
    ms_token = max_over_ranks(run_token_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream))
    token_launches = (dec.kl_launch_count() - l0t - 1) / (K + W)
    # 2d. the K timed tokens in one launch (kl_decode_greedy_tokens)
    l0k = dec.kl_launch_count()
    ms_tokens = max_over_ranks(run_tokens_per_launch(dec, fresh_cache(), tok0, context, W, K, stream))
    tokens_launches = dec.kl_launch_count() - l0k - 1 - W
    # 2b. both schedules again with one step captured in a CUDA graph (no per-launch host cost): the per-layer
    #     baseline at its best, so that the looped kernel is not compared with a strawman
    graph_ms, graph_err = {}, {}
    for name, mode in (("looped", binding.KL_MODE_LOOPED), ("per_layer", binding.KL_MODE_PER_LAYER),
                       ("per_stage", binding.KL_MODE_PER_STAGE)):
        dec.kl_set_mode(mode)
        ms, err = run_graph_loop(dec, fresh_cache(), tok0, context, batch, W, K)
        graph_ms[name] = max_over_ranks(ms) if ms is not None and not _DIST["on"] else ms
        graph_err[name] = err
    ms, err = run_graph_loop(dec, fresh_cache(), tok0, context, batch, W, K, greedy=True)
    graph_ms["one_launch_per_token"] = max_over_ranks(ms) if ms is not None and not _DIST["on"] else ms
    graph_err["one_launch_per_token"] = err
    # 3. roofline of the dominant kernel: events around the decoder launch inside the timed steps
    dec.kl_set_mode(binding.KL_MODE_LOOPED)
    dec.kl_profile_enable(K)
    run_device_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream)
    dec_ms, cls_ms = dec.kl_profile_read(K)
    dec.kl_profile_enable(0)
    clocks = sampler.stop()
    # 4. end to end through the host-buffer entry point
    ms_e2e_logits = max_over_ranks(run_host_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream))
    ms_e2e = max_over_ranks(run_greedy_host_loop(dec, fresh_cache(), tok0, context, batch, W, K, stream))
    ms_e2e_tokens = max_over_ranks(run_tokens_per_launch(dec, fresh_cache(), tok0, context, W, K, stream, host=True))
    # 5. where the model runs in stash mode: the same tokens in the plain mode (a second handle with KL_FLAG_NO_STASH),
    #    if both copies of the weights fit the device
    stash_mode = dec.kl_stash_mode()
    plain = None
    free_b, _ = torch.cuda.mem_get_info()
    fits = free_b > dec.weight_bytes + dec.scratch_bytes + cache.numel() * 2 + (4 << 30)
    fits = max_over_ranks(0.0 if fits else 1.0) == 0.0   # the same decision on every replica: the passes below synchronise them
    if stash_mode == 1 and batch == 1 and fits:
        dec2, cache2, _ = build_model(shape, batch, context, 2 * (K + W), seed=rank, stash=False)
        ms_p_token = max_over_ranks(run_token_loop(dec2, cache2, tok0, context, batch, W, K, stream))
        dec2.kl_set_mode(binding.KL_MODE_LOOPED)
        cache2, = (gen.make_kv_cache(shape, batch, context, context + 2 * (K + W) + 8, rank, "cuda"),)
        ms_p_looped = max_over_ranks(run_device_loop(dec2, cache2, tok0, context, batch, W, K, stream))
        plain = {"one_launch_per_token": {"value": K * batch * world / (ms_p_token * 1e-3), "ms_per_step": ms_p_token / K},
                 "looped_four_launches": {"value": K * batch * world / (ms_p_looped * 1e-3), "ms_per_step": ms_p_looped / K},
                 "what": "the same model created with KL_FLAG_NO_STASH: weights consumed from the shared-memory ring"}
        dec2.close()
        del dec2, cache2

    tokens = K * batch * world
    # headline: the schedule with the fewest calls -- the K timed tokens decoded by ONE call of kl_decode_greedy_tokens (the
    # loop over layers extended to a loop over tokens: decoder layers, classifier and sampling of up to 256 tokens per
    # launch of the persistent kernel); one launch per token, the four-launch looped schedule and the boundary
    # schedules are reported beside it
    ms_head = ms_tokens
    head_launches = max(1, (K + 255) // 256)   # launches of kl_token_kernel in the timed call
    value = tokens / (ms_head * 1e-3)   # already the maximum over the replicas
    pos_avg = context + W + (K - 1) / 2.0
    bytes_step = step_bytes(shape, batch, 0) + kv_bytes(shape, batch, 0) * pos_avg  # kv_bytes(.,.,0) = one row set
    # one decoder launch decodes ONE sequence (batches run sequence after sequence): its algorithmic bytes are one
    # sequence's; bytes_step stays the batched step's (weights once), so for batch > 1 the whole-step fractions show how
    # far the sequential schedule is from the batched roofline
    bytes_dec = decoder_bytes(shape, 1, 0) + kv_bytes(shape, 1, 0) * pos_avg
    peaks = measured_peaks()
    dec_avg_ms = statistics.mean(dec_ms)
    achieved = bytes_dec / (dec_avg_ms * 1e-3) / 1e9
    line = {
        "metric": "decode tokens/s", "value": value, "unit": "tokens/s", "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_head / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": args.workload, "batch": batch, "context": context, "l2": "inputs larger than L2 (weights and KV streamed once per step)"},
        "details": {"mode": "looped over layers and tokens (kl_decode_greedy_tokens: decoder layers + classifier + sampling of "
                            "the K timed tokens in one call, up to 256 tokens per launch)",
                    "storage": "bf16 weights and KV, fp32 activations and accumulation",
                    "stash_mode": stash_mode,
                    "parallelism": "replicas only" if world > 1 else "single GPU",
                    "batch_schedule": "one sequence after another (weights streamed once per sequence)" if batch > 1 else "n/a",
                    "max_ctx": max_ctx},
        "clocks": clocks, "gpu_launches": int(tokens_launches),
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 8 * batch,
                "d2h_bytes_per_step": 4 * batch, "call": "kl_decode_greedy_host (tokens and positions in, next tokens out)"},
        "e2e_logits": {"value": tokens / (ms_e2e_logits * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 8 * batch,
                       "d2h_bytes_per_step": 4 * shape.vocab * batch,
                       "call": "kl_decode_step_host (logits copied back, the host picks the next token)"},
        # the dominant (only) kernel of the timed region: one launch = one step = all bytes of the step
        "roofline": {"bound": "hbm", "kernel": "kl_token_kernel (all layers + classifier + sampling of every token of the launch; "
                                               "%d token(s) per launch in the timed call)" % (K // head_launches),
                     "achieved": bytes_step / (ms_head / K * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": bytes_step / (ms_head / K * 1e-3) / 1e9 / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "traffic": ((ncu_traffic(shape, batch, context) + NCU_DRAM_BYTES_CLASSIFIER_STAGE_V128256_H4096) * K / head_launches
                                 if ncu_traffic(shape, batch, context) and (shape.vocab, shape.hidden) == (128256, 4096) else None),
                     "traffic_source": "ncu dram bytes read+written of a 4-layer kl_token_kernel launch: its decoder layers (the "
                                       "4-layer kl_decoder_kernel capture) scaled by layers/4, its classifier and sampling stages "
                                       "(the difference of the two captures) once "
                                       "(profiles/kl_token_kernel_llama31_8b_4layers_b1_ctx4096.txt, "
                                       "profiles/kl_decoder_kernel_llama31_8b_4layers_b1_ctx4096.txt)",
                     "bytes_per_launch": bytes_step * K / head_launches, "ms_per_launch": ms_head / head_launches},
        "looped_four_launches": {"value": tokens / (ms_looped * 1e-3), "ms_per_step": ms_looped / K,
                                 "launches_per_step": int(launches) // K},
        "decoder_kernel": {"bound": "hbm", "kernel": "kl_decoder_kernel (looped, all layers; events inside the four-launch schedule)", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": peaks["source"], "traffic": ncu_traffic(shape, batch, context),
                     "traffic_source": ("ncu dram bytes read+written of a 4-layer launch, scaled by layers/4 "
                                        "(profiles/kl_decoder_kernel_llama31_8b_4layers_b1_ctx4096.txt)"
                                        if ncu_traffic(shape, batch, context) else None),
                     "bytes_per_launch": bytes_dec,
                     "ms_per_launch": dec_avg_ms, "classifier_ms": statistics.mean(cls_ms)},
        "whole_step": {"bytes_per_step": bytes_step, "gbs": bytes_step / (ms_head / K * 1e-3) / 1e9,
                       "frac_of_measured_copy": bytes_step / (ms_head / K * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       "frac_of_8tbs": bytes_step / (ms_head / K * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
        "cuda_graph": {k: ({"value": tokens / (graph_ms[k] * 1e-3), "ms_per_step": graph_ms[k] / K} if graph_ms[k]
                           else {"value": None, "why": graph_err[k]}) for k in graph_ms},
        "per_stage": {"value": tokens / (ms_stage * 1e-3), "ms_per_step": ms_stage / K,
                      "launches_per_step": 5 * shape.n_layers + 3, "looped_speedup": ms_stage / ms_looped},
        "one_launch_per_token": {"value": tokens / (ms_token * 1e-3), "ms_per_step": ms_token / K,
                                 "launches_per_step": token_launches, "vs_four_launches": ms_looped / ms_token},
        "tokens_per_launch": {"value": tokens / (ms_tokens * 1e-3), "ms_per_step": ms_tokens / K, "launches": tokens_launches,
                              "call": "kl_decode_greedy_tokens: the K timed tokens in one call (up to 256 tokens per launch)",
                              "e2e": {"value": tokens / (ms_e2e_tokens * 1e-3), "h2d_bytes_per_call": 8, "d2h_bytes_per_call": 4 * K,
                                      "call": "kl_decode_greedy_tokens_host, host clock"}},
        "per_layer": {"value": tokens / (ms_layer * 1e-3), "ms_per_step": ms_layer / K,
                      "launches_per_step": shape.n_layers + 3,
                      "looped_speedup": ms_layer / ms_looped},
    }
    if plain is not None:
        line["plain_mode"] = plain
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import kl_oracle as ko
        ko.build()
        # whole decode steps where the host holds the model (up to the 8B shape), otherwise a bounded sample of up to 8
        # layers + the classifier; repeated until about 12 s of CPU work
        smp = OracleSampler(shape, batch, context, oracle_layers_that_fit(shape) or min(8, shape.n_layers))
        secs = [smp.step()]
        t_exec = smp.t_layers + smp.t_cls
        while len(secs) < 40 and t_exec * (len(secs) + 1) < 12.0:
            secs.append(smp.step())
        sec = statistics.mean(secs)
        line["cpu_baseline"] = {"value": 1.0 / sec, "unit": "tokens/s", "cores": smp.threads, "kind": "oracle",
                                "sample": smp.describe() + f"; mean of {len(secs)} such executions"}
    dec.close()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_ours_batched(args, shape, batch, context):
    """Workloads with batch > 1: the tensor-core path (one dense contraction per projection for the whole batch,
    weights streamed once per step) is the headline; the same batch decoded sequence after sequence by the looped
    batch-1 kernel is timed beside it."""
    from paper_2410_23668_b200 import binding, build
    if build.needs_build():
        build.build_library()
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        torch.distributed.init_process_group("nccl", device_id=torch.device("cuda", local))
        _DIST["on"] = True
    K, W = args.steps, max(args.warmup, 3)
    Ks = max(1, min(K, 4))   # the sequential schedule takes batch times longer per step: fewer steps
    dec, cache, max_ctx = build_model(shape, batch, context, 9 * (K + W) + Ks + 3, seed=rank)
    tok0 = gen.make_tokens(shape, batch, rank, device="cuda")
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local)
    sampler.start()
    # the cache is not restored between the passes: the rows the passes append lie beyond the positions they read
    dec.kl_set_batched_path(True)
    # the three call schedules of the batched step, from the same phase code (Section 2 of the paper, schedules
    # (iii), (ii), (i)): one cooperative launch per step, that kernel launched per layer, one launch per operator group
    dec.kl_set_mode(binding.KL_MODE_LOOPED)
    l0 = dec.kl_launch_count()
    ms_looped = max_over_ranks(run_device_loop(dec, cache, tok0, context, batch, W, K, stream))
    looped_launches = (dec.kl_launch_count() - l0) // (K + W)
    dec.kl_set_mode(binding.KL_MODE_PER_LAYER)
    l0 = dec.kl_launch_count()
    ms_layer = max_over_ranks(run_device_loop(dec, cache, tok0, context, batch, W, K, stream))
    layer_launches = (dec.kl_launch_count() - l0) // (K + W)
    dec.kl_set_mode(binding.KL_MODE_PER_STAGE)   # the fastest of the three on this GPU, and the default for batches
    l0 = dec.kl_launch_count()
    ms_batched = max_over_ranks(run_device_loop(dec, cache, tok0, context, batch, W, K, stream))
    launches = (dec.kl_launch_count() - l0) * K // (K + W)
    # the same greedy steps through kl_decode_greedy: the library replays the step from the CUDA graph it keeps
    ms_greedy = max_over_ranks(run_token_loop(dec, cache, tok0, context, batch, W, K, stream))
    ms_graph, graph_err = run_graph_loop(dec, cache, tok0, context, batch, W, K)
    if ms_graph is not None and _DIST["on"]:
        ms_graph = max_over_ranks(ms_graph)
    dec.kl_profile_enable(K)
    run_device_loop(dec, cache, tok0, context, batch, W, K, stream)
    dec_ms, cls_ms = dec.kl_profile_read(K)
    dec.kl_profile_enable(0)
    clocks = sampler.stop()
    ms_e2e_logits = max_over_ranks(run_host_loop(dec, cache, tok0, context, batch, W, K, stream))
    ms_e2e = max_over_ranks(run_greedy_host_loop(dec, cache, tok0, context, batch, W, K, stream))
    # the same launches in plain stream order (no programmatic dependent launch): what the launch boundaries cost
    dec.kl_set_dependent_launch(False)
    ms_plain = max_over_ranks(run_device_loop(dec, cache, tok0, context, batch, W, K, stream))
    dec.kl_set_dependent_launch(True)
    dec.kl_set_batched_path(False)
    dec.kl_set_mode(binding.KL_MODE_LOOPED)   # the batch-1 looped kernel, sequence after sequence
    ms_seq = max_over_ranks(run_device_loop(dec, cache, tok0, context, batch, 3, Ks, stream))

    tokens = K * batch * world
    pos_avg = context + W + (K - 1) / 2.0
    bytes_step = step_bytes(shape, batch, 0) + kv_bytes(shape, batch, 0) * pos_avg
    bytes_dec = decoder_bytes(shape, batch, 0) + kv_bytes(shape, batch, 0) * pos_avg
    peaks = measured_peaks()
    dec_avg_ms = statistics.mean(dec_ms)
    achieved = bytes_dec / (dec_avg_ms * 1e-3) / 1e9
    line = {
        # headline: greedy decoding through kl_decode_greedy (the step replayed from the library's own CUDA graph)
        "metric": "decode tokens/s", "value": tokens / (ms_greedy * 1e-3), "unit": "tokens/s", "n_gpus": world, "steps": K,
        "warmup": W, "ms_per_step": ms_greedy / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": args.workload, "batch": batch, "context": context, "l2": "inputs larger than L2 (weights and KV streamed once per step)"},
        "details": {"mode": "batched tensor-core path, kl_decode_greedy chained on the device",
                    "storage": "bf16 weights and KV; fp32 activations enter the tcgen05 MMAs as two bf16 halves, fp32 accumulation",
                    "parallelism": "replicas only" if world > 1 else "single GPU",
                    "batch_schedule": "all sequences per launch (weights streamed once per step)",
                    "max_ctx": max_ctx},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": tokens / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 8 * batch,
                "d2h_bytes_per_step": 4 * batch, "call": "kl_decode_greedy_host (tokens and positions in, next tokens out)"},
        "e2e_logits": {"value": tokens / (ms_e2e_logits * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": 8 * batch,
                       "d2h_bytes_per_step": 4 * shape.vocab * batch,
                       "call": "kl_decode_step_host (logits copied back, the host picks the next token)"},
        "roofline": {"bound": "hbm", "kernel": "all launches of the decoder layers (kl_bgemm_kernel x4, kl_b_attn_kernel and "
                                               "the vector kernels, per layer)", "achieved": achieved,
                     "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": peaks["source"], "traffic": ncu_traffic(shape, batch, context),
                     "traffic_source": ("ncu dram bytes read+written of the ten launches of one layer, scaled by the layer count "
                                        "(profiles/batched_path_llama31_8b_2layers_b32_ctx4096.txt)"
                                        if ncu_traffic(shape, batch, context) else None),
                     "bytes_per_launch": bytes_dec,
                     "ms_per_launch": dec_avg_ms, "classifier_ms": statistics.mean(cls_ms)},
        "whole_step": {"bytes_per_step": bytes_step, "gbs": bytes_step / (ms_greedy / K * 1e-3) / 1e9,
                       "frac_of_measured_copy": bytes_step / (ms_greedy / K * 1e-3) / 1e9 / peaks["hbm_gbs"],
                       "frac_of_8tbs": bytes_step / (ms_greedy / K * 1e-3) / 1e9 / NOMINAL_HBM_GBS},
        "cuda_graph": ({"value": tokens / (ms_graph * 1e-3), "ms_per_step": ms_graph / K} if ms_graph
                       else {"value": None, "why": graph_err}),
        "launch_by_launch": {"value": tokens / (ms_batched * 1e-3), "ms_per_step": ms_batched / K,
                             "call": "kl_decode_step + kl_argmax_advance, every kernel launched from the host (dependent launch on)"},
        "looped": {"value": tokens / (ms_looped * 1e-3), "ms_per_step": ms_looped / K, "launches_per_step": looped_launches,
                   "what": "KL_MODE_LOOPED: one persistent kernel per step (grid barriers between the phases, weight stream running ahead)"},
        "per_layer": {"value": tokens / (ms_layer * 1e-3), "ms_per_step": ms_layer / K, "launches_per_step": layer_launches,
                      "looped_speedup": ms_layer / ms_looped},
        "per_stage": {"value": tokens / (ms_batched * 1e-3), "ms_per_step": ms_batched / K, "launches_per_step": int(launches) // K,
                      "looped_speedup": ms_batched / ms_looped},
        "plain_stream_order": {"value": tokens / (ms_plain * 1e-3), "ms_per_step": ms_plain / K,
                               "launches_per_step": int(launches) // K},
        "sequential_looped": {"value": Ks * batch * world / (ms_seq * 1e-3), "ms_per_step": ms_seq / Ks, "steps": Ks,
                              "batched_speedup": (ms_seq / Ks) / (ms_greedy / K)},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import kl_oracle as ko
        ko.build()
        smp = OracleSampler(shape, batch, context, (oracle_layers_that_fit(shape) or 1) if batch * context <= 16384 else 1)
        secs = [smp.step()]
        t_exec = smp.t_layers + smp.t_cls
        while len(secs) < 40 and t_exec * (len(secs) + 1) < 12.0:
            secs.append(smp.step())
        sec = statistics.mean(secs)
        line["cpu_baseline"] = {"value": 1.0 / sec, "unit": "tokens/s", "cores": smp.threads, "kind": "oracle",
                                "sample": smp.describe() + f"; mean of {len(secs)} such executions"}
    dec.close()
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of one looped launch over 4 layers of the 8B shape at batch 1,
# context 4096 (ncu capture summarised under profiles/), per layer.  Every layer streams its own weights and KV once,
# so a full launch is this times the layer count.
NCU_DRAM_BYTES_PER_LAYER_8B_B1_CTX4096 = (1.814647e9 + 20.904704e6) / 4


# the same for the ten launches of one layer of the batched path at batch 32, context 4096
NCU_DRAM_BYTES_PER_LAYER_8B_B32_CTX4096 = 1000.9e6


# dram bytes of the classifier and sampling stages of kl_token_kernel at vocabulary 128256, hidden 4096: a 4-layer
# kl_token_kernel launch minus a 4-layer kl_decoder_kernel launch (both captures summarised under profiles/)
NCU_DRAM_BYTES_CLASSIFIER_STAGE_V128256_H4096 = (2.864009e9 + 22.105344e6) - (1.814647e9 + 20.904704e6)


def ncu_traffic(shape, batch, context):
    """Bytes per looped launch (batch 1) or per step's decoder layers (batch 32), from the committed ncu captures; None
    for workloads that were not captured."""
    if batch == 32 and context == 4096 and (shape.hidden, shape.ffn, shape.n_q_heads, shape.n_kv_heads, shape.head_dim) == \
            (4096, 14336, 32, 8, 128):
        return NCU_DRAM_BYTES_PER_LAYER_8B_B32_CTX4096 * shape.n_layers
    if batch == 1 and context == 4096 and (shape.hidden, shape.ffn, shape.n_q_heads, shape.n_kv_heads, shape.head_dim) == \
            (4096, 14336, 32, 8, 128):
        return NCU_DRAM_BYTES_PER_LAYER_8B_B1_CTX4096 * shape.n_layers
    return None


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    shape, batch, context, dsteps = WORKLOADS[args.workload]
    if args.steps is None:
        args.steps = dsteps
    if args.impl == "reference":
        run_reference(args, shape, batch, context)
    else:
        (run_ours if batch == 1 else run_ours_batched)(args, shape, batch, context)


if __name__ == "__main__":
    main()
