"""Parity of the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs.
Tolerances: rel-L2 <= 1e-2 on hidden state and logits, max |delta logit| <= 5e-2, identical greedy tokens
(teacher-forced), looped == per-layer bit for bit."""
import numpy as np
import pytest
import torch

from paper_2410_23668_b200 import binding, inputs as gen
from tests import helpers

pytestmark = pytest.mark.gpu


def test_generator_is_bit_identical_on_cpu_and_cuda():
    for name in ("wq", "wdown", "norm1"):
        a = gen.make_tensor(gen.TINY, name, 1, 5, "cpu")
        b = gen.make_tensor(gen.TINY, name, 1, 5, "cuda").cpu()
        assert torch.equal(a, b)
    a = gen.make_kv_cache(gen.TINY, 1, 33, 40, 2, "cpu")
    b = gen.make_kv_cache(gen.TINY, 1, 33, 40, 2, "cuda").cpu()
    assert torch.equal(a, b)


def test_tiny_16_greedy_steps_all_schedules():
    """Config 1: 4 layers, hidden 256, 4/2 heads of 64, FFN 512, vocab 1024, 128 cached positions, 16 steps."""
    rep = helpers.run_parity(gen.TINY, context=128, steps=16, seed=0)
    helpers.assert_parity(rep, 16)


@pytest.mark.parametrize("context", [0, 1, 63, 64, 65, 700])
def test_ragged_contexts(context):
    """Empty cache (the new token attends to itself only), one cached position, chunk-boundary lengths, several
    split-K chunks with a ragged tail."""
    rep = helpers.run_parity(gen.TINY, context=context, steps=3, seed=1)
    helpers.assert_parity(rep, 3)


SHAPES = {
    # rows not divisible by the CTA count or the tile sizes, head_dim 128, G = 4
    "odd_rows_hd128": gen.ModelShape(3, 328, 8, 2, 128, 1000, 1544, 1e-5, 500000.0),
    # FFN wider than one ring slot: down-projection rows are split into pieces merged in shared memory
    "split_k_down": gen.ModelShape(2, 64, 2, 1, 32, 9000, 520, 1e-5, 10000.0),
    # hidden = 8192: a (gate, up) pair no longer fits one slot, the pair spans two chunks; G = 8
    "wide_hidden_g8": gen.ModelShape(2, 8192, 8, 1, 64, 264, 520, 1e-5, 500000.0),
    # G = 1 (multi-head attention), head_dim 256
    "mha_hd256": gen.ModelShape(2, 512, 2, 2, 256, 768, 1000, 1e-6, 10000.0),
}


@pytest.mark.parametrize("name", sorted(SHAPES))
def test_odd_shapes(name):
    rep = helpers.run_parity(SHAPES[name], context=150, steps=3, seed=3)
    helpers.assert_parity(rep, 3)


# Shapes that take the stash mode (weights through tensor memory) on paths the 8B shape does not use: rows of 2048
# columns (four rows per chunk, two units per group) and a down projection of two pieces of 4096 columns.
STASH_SHAPES = {
    "rows_of_2048": gen.ModelShape(2, 2048, 16, 4, 128, 4096, 1544, 1e-5, 500000.0),
    "down_in_two_pieces": gen.ModelShape(2, 4096, 32, 8, 128, 8192, 1544, 1e-5, 500000.0),
    # one layer, a classifier of 50 units for 148 CTAs (most CTAs stream nothing in that stage), rows of 3072 columns
    # (three granules per row: two granules of every chunk stay unused), G = 3
    "few_units_rows_of_3072": gen.ModelShape(1, 3072, 24, 8, 128, 1024, 200, 1e-5, 500000.0),
    # chunks of 1024 columns, eight rows each (FFN 5120 = 5 x 1024)
    "pieces_of_1024": gen.ModelShape(2, 2048, 16, 4, 128, 5120, 1544, 1e-5, 500000.0),
}


@pytest.mark.parametrize("name", sorted(STASH_SHAPES))
def test_stash_mode_shapes(name):
    rep = helpers.run_parity(STASH_SHAPES[name], context=300, steps=3, seed=5)
    assert rep["stash_mode"] == 1
    helpers.assert_parity(rep, 3)


def test_llama31_8b_layer_shape_both_modes():
    """The 8B layer shape (two layers) in stash mode and with KL_FLAG_NO_STASH: both match the oracle, and the odd shapes
    above never take the stash mode."""
    import dataclasses
    shape = dataclasses.replace(gen.LLAMA31_8B, n_layers=2)
    for stash in (True, False):
        rep = helpers.run_parity(shape, context=700, steps=3, seed=2, stash=stash)
        assert rep["stash_mode"] == (1 if stash else 0)
        helpers.assert_parity(rep, 3)
    rep = helpers.run_parity(SHAPES["odd_rows_hd128"], context=20, steps=1, seed=1)
    assert rep["stash_mode"] == 0


def test_llama31_8b_shape_16_greedy_steps():
    """Config 2: Llama-3.1-8B shape, batch 1, context 4096, first 16 decode steps, looped and per-layer."""
    rep = helpers.run_parity(gen.LLAMA31_8B, context=4096, steps=16, seed=0, max_ctx=4096 + 136, check_cache=False)
    helpers.assert_parity(rep, 16, check_cache=False)
    margins = [r["margin"][0] for r in rep["ref"]]
    print("oracle top-1/top-2 logit margins:", ["%.3f" % m for m in margins])


def test_llama31_8b_shape_context_65536():
    """Config 3 by sampled layers: the 8B shape at context 65536 (attention-heavy: every split-K unit streams ~3640
    positions), the first two layers and the classifier, two decode steps.  The oracle streams the same layers."""
    import dataclasses
    shape = dataclasses.replace(gen.LLAMA31_8B, n_layers=2)
    rep = helpers.run_parity(shape, context=65536, steps=2, seed=0, max_ctx=65536 + 8, check_cache=False)
    helpers.assert_parity(rep, 2, check_cache=False)


def test_llama31_70b_shape_two_layers():
    """Config 5 by sampled layers: the 70B shape (hidden 8192, 64 / 8 heads, FFN 28672) at context 4096, the first two
    layers and the classifier, two decode steps."""
    import dataclasses
    shape = dataclasses.replace(gen.LLAMA31_70B, n_layers=2)
    rep = helpers.run_parity(shape, context=4096, steps=2, seed=0, max_ctx=4096 + 8, check_cache=False)
    helpers.assert_parity(rep, 2, check_cache=False)


def test_batch_of_sequences_ragged_positions():
    """Without the batched path a batch is decoded one sequence after another by the batch-1 kernels: three sequences
    at different positions, four steps, all schedules; every sequence matches the oracle and its cache rows land in
    its own slab of the [L][2][B][nkv][max_ctx][hd] cache."""
    rep = helpers.run_parity(gen.TINY, context=128, steps=4, seed=3, batch=3, positions0=[5, 64, 128], batched_path=False)
    helpers.assert_parity(rep, 4, batch=3)


BATCHED = {
    # name: (shape, batch, context, first positions)
    "tiny_b3": (gen.TINY, 3, 128, [5, 64, 128]),
    # a full batch with every length from an empty cache up: attention units with no position, one position, ragged tails
    "tiny_b32": (gen.TINY, 32, 330, [0, 1, 2, 31, 32, 33, 63, 64, 65, 127, 128, 129] + list(range(130, 330, 10))),
    # rows and columns that are no multiples of the 128 x 64 tiles (TMA fills the tile edges with zeros), head size 128
    "odd_rows_hd128_b5": (SHAPES["odd_rows_hd128"], 5, 150, [0, 17, 64, 149, 150]),
    # gate/up stored in chunk order (units of two rows cut into two column pieces): the rank-5 / rank-4 tensor maps; G = 8
    "wide_hidden_g8_b4": (SHAPES["wide_hidden_g8"], 4, 150, [3, 77, 128, 150]),
}


@pytest.mark.parametrize("name", sorted(BATCHED))
def test_batched_tensor_core_path(name):
    """Batches on the tcgen05 path (every projection one dense contraction for the whole batch; the default for
    batch > 1): every sequence matches the oracle within the same tolerances as the batch-1 kernels, greedy tokens
    included, and the appended cache rows land in the right slabs.

    The projections take their fp32 inputs as two bf16 halves (16 significant bits instead of 24), so a k or v value
    that lies within ~2^-17 of a bf16 rounding boundary may round the other way than in the oracle; for a sequence
    with a single cached position that one-step difference reaches the next layer undiluted and flips more there.
    Every appended value is still within one bf16 step of the oracle's (checked); only the share of values that
    differ at all is allowed to be larger than for the fp32 batch-1 kernels."""
    shape, batch, context, pos0 = BATCHED[name]
    # the three schedules of the batched step -- the looped kernel (one launch per step), the same kernel launched per
    # layer, one launch per operator group -- run the same phase code: identical bits
    rep = helpers.run_parity(shape, context=context, steps=3, seed=3, batch=batch, positions0=pos0, batched_path=True)
    helpers.assert_parity(rep, 3, batch=batch, flip_tol=0.05)


def test_batched_path_llama31_8b_shape_b32():
    """Config 4 by sampled layers: the 8B shape (down projection in chunk order with ten column pieces), batch 32,
    ragged contexts up to 1024, the first two layers and the classifier, two decode steps."""
    import dataclasses
    shape = dataclasses.replace(gen.LLAMA31_8B, n_layers=2)
    pos0 = [1024 - 29 * i for i in range(32)]
    rep = helpers.run_parity(shape, context=1024, steps=2, seed=0, batch=32, positions0=pos0, max_ctx=1024 + 8,
                             batched_path=True, check_cache=False)
    helpers.assert_parity(rep, 2, batch=32, check_cache=False)


def test_batched_path_llama31_8b_full_depth():
    """All 32 layers of the 8B shape on the batched path (the layer coordinate of every tensor map, the residual
    stream carried through 128 projections), four sequences with ragged contexts up to 512, two decode steps."""
    pos0 = [512, 300, 77, 0]
    rep = helpers.run_parity(gen.LLAMA31_8B, context=512, steps=2, seed=0, batch=4, positions0=pos0, max_ctx=512 + 8,
                             modes=(binding.KL_MODE_LOOPED,), batched_path=True, check_cache=False, stream_layers=True)
    helpers.assert_parity(rep, 2, batch=4, check_cache=False)


def test_batched_path_llama31_70b_shape_b8():
    """The 70B layer shape (hidden 8192: gate/up in chunk order with two column pieces, down with twenty) at batch 8,
    ragged contexts up to 2048, the first two layers and the classifier, two decode steps."""
    import dataclasses
    shape = dataclasses.replace(gen.LLAMA31_70B, n_layers=2)
    pos0 = [2048, 1500, 1024, 777, 300, 64, 1, 0]
    rep = helpers.run_parity(shape, context=2048, steps=2, seed=0, batch=8, positions0=pos0, max_ctx=2048 + 8,
                             modes=(binding.KL_MODE_LOOPED,), batched_path=True, check_cache=False)
    helpers.assert_parity(rep, 2, batch=8, check_cache=False)


# Decoder shape of the 3B model of the paper's Table 2 (public hyper-parameters: 28 layers, hidden 3072, 24 query and
# 8 kv heads of 128, FFN 8192); two layers of it here.
LLAMA32_3B_2L = gen.ModelShape(2, 3072, 24, 8, 128, 8192, 128256, 1e-5, 500000.0)


def test_llama32_3b_shape_two_layers():
    """A second decoder shape by its dimensions (G = 3 query heads per kv head, hidden 3072): the batch-1 kernel in its
    three schedules, context 2048, two steps."""
    rep = helpers.run_parity(LLAMA32_3B_2L, context=2048, steps=2, seed=0, max_ctx=2048 + 8, check_cache=False)
    helpers.assert_parity(rep, 2, check_cache=False)


def test_batched_path_llama32_3b_shape_b16():
    """The same shape on the batched path: 16 sequences, ragged contexts up to 2048, two steps."""
    pos0 = [2048 - 131 * i for i in range(16)]
    rep = helpers.run_parity(LLAMA32_3B_2L, context=2048, steps=2, seed=0, batch=16, positions0=pos0, max_ctx=2048 + 8,
                             modes=(binding.KL_MODE_LOOPED,), batched_path=True, check_cache=False)
    helpers.assert_parity(rep, 2, batch=16, check_cache=False)


def test_qwen25_72b_shape_two_layers_both_paths():
    """The 72B decoder of the paper's Table 2 by its public dimensions (hidden 8192, 64 / 8 heads of 128, FFN 29568,
    vocabulary 152064, biases on q, k, v), two layers: the looped batch-1 kernel and the batched path, two steps."""
    shape = gen.ModelShape(2, 8192, 64, 8, 128, 29568, 152064, 1e-6, 1000000.0, True)
    rep = helpers.run_parity(shape, context=1024, steps=2, seed=0, max_ctx=1024 + 8, check_cache=False,
                             modes=(binding.KL_MODE_LOOPED, binding.KL_MODE_PER_LAYER))
    helpers.assert_parity(rep, 2, check_cache=False)
    rep = helpers.run_parity(shape, context=1024, steps=2, seed=0, batch=4, positions0=[1024, 700, 33, 0], max_ctx=1024 + 8,
                             modes=(binding.KL_MODE_LOOPED,), batched_path=True, check_cache=False)
    helpers.assert_parity(rep, 2, batch=4, check_cache=False)


def test_qkv_bias_both_paths():
    """A decoder whose q, k, v projections carry biases (flag KL_FLAG_QKV_BIAS, tensors bq / bk / bv): the batch-1 kernel
    in its three schedules and the batched path against the oracle; and the flag is checked -- a model without it
    refuses bias tensors, a model with it does not run before they are loaded."""
    import dataclasses
    shape = dataclasses.replace(gen.TINY, qkv_bias=True)
    rep = helpers.run_parity(shape, context=128, steps=4, seed=5)
    helpers.assert_parity(rep, 4)
    rep = helpers.run_parity(shape, context=128, steps=3, seed=5, batch=5, positions0=[0, 17, 64, 127, 128],
                             modes=(binding.KL_MODE_LOOPED,), batched_path=True)
    helpers.assert_parity(rep, 3, batch=5, flip_tol=0.05)
    wide = dataclasses.replace(LLAMA32_3B_2L, qkv_bias=True)   # head size 128, G = 3
    rep = helpers.run_parity(wide, context=300, steps=2, seed=5, max_ctx=308, check_cache=False)
    helpers.assert_parity(rep, 2, check_cache=False)
    dec = binding.Decoder(gen.TINY, 1, 64)
    with pytest.raises(binding.KlError) as e:
        dec.kl_load_weights("bq", 0, torch.zeros(gen.TINY.q_dim, dtype=torch.bfloat16, device="cuda"))
    assert e.value.code == binding.KL_ERR_INVALID_ARG
    dec.close()
    dec = binding.Decoder(shape, 1, 64)
    for l in range(shape.n_layers):
        for name, t in gen.make_layer(gen.TINY, l, 0, "cuda").items():   # everything but the biases
            dec.kl_load_weights(name, l, t)
    for name, t in gen.make_globals(shape, 0, "cuda").items():
        dec.kl_load_weights(name, -1, t)
    cache = gen.make_kv_cache(shape, 1, 8, 64, 0, "cuda")
    with pytest.raises(binding.KlError) as e:
        dec.kl_decode_step(torch.zeros(1, dtype=torch.int32, device="cuda"), torch.full((1,), 8, dtype=torch.int32, device="cuda"),
                           cache, torch.empty(1, shape.vocab, device="cuda"), 1)
    assert e.value.code == binding.KL_ERR_NOT_LOADED
    dec.close()


def test_batched_path_is_reproducible_and_optional():
    """The partial results are added in a fixed order: the same batched step again gives identical bits, with and
    without programmatic dependent launch.  A shape without
    the path (head size 32) refuses to switch it on and decodes batches on the batch-1 kernels."""
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 4, 200, 0)
    cache0 = gen.make_kv_cache(shape, 4, 128, 200, 0, "cuda")
    tok = gen.make_tokens(shape, 4, 0).cuda()
    pos = torch.tensor([128, 7, 64, 0], dtype=torch.int32, device="cuda")
    outs = []
    for run in range(4):
        dec.kl_set_dependent_launch(run < 3)   # the last run in plain stream order: same kernels, same bits
        cache = cache0.clone()
        logits = torch.empty(4, shape.vocab, device="cuda")
        hidden = torch.empty(4, shape.hidden, device="cuda")
        dec.kl_decode_step(tok, pos, cache, logits, 4)
        dec.kl_read_hidden(hidden, 4)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        outs.append((logits.cpu(), hidden.cpu(), cache.cpu().view(torch.uint16)))
    for lg, hd, ch in outs[1:]:
        assert torch.equal(lg, outs[0][0]) and torch.equal(hd, outs[0][1]) and torch.equal(ch, outs[0][2])
    dec.close()
    dec = binding.Decoder(SHAPES["split_k_down"], 2, 64)
    with pytest.raises(binding.KlError) as e:
        dec.kl_set_batched_path(True)
    assert e.value.code == binding.KL_ERR_UNSUPPORTED_SHAPE
    dec.kl_set_batched_path(False)
    dec.close()


@pytest.mark.parametrize("batched", [True, False])
def test_batch_bad_entry_makes_the_whole_step_a_no_op(batched):
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 2, 200, 0)
    dec.kl_set_batched_path(batched)
    cache = gen.make_kv_cache(shape, 2, 128, 200, 0, "cuda")
    before = cache.clone()
    tok = torch.tensor([1, shape.vocab + 7], dtype=torch.int32, device="cuda")   # the SECOND sequence is bad
    pos = torch.tensor([128, 128], dtype=torch.int32, device="cuda")
    logits = torch.full((2, shape.vocab), 7.0, device="cuda")
    dec.kl_decode_step(tok, pos, cache, logits, 2)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_ERR_OUT_OF_RANGE
    assert torch.equal(cache.view(torch.uint16), before.view(torch.uint16))       # nothing appended, not even for sequence 0
    assert bool((logits == 7.0).all())
    # the handle stays usable: the same step with valid tokens runs
    tok[1] = 2
    dec.kl_decode_step(tok, pos, cache, logits, 2)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    assert bool(torch.isfinite(logits).all()) and not bool((logits == 7.0).all())
    dec.close()


def test_captured_step_replays_like_plain_launches():
    """One decode step + sampling captured in a CUDA graph and replayed gives the same tokens and logits as the same
    steps launched one by one: nothing in a step depends on host state that a replay would not advance (the step
    counter behind the tags lives on the device)."""
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 1, 200, 0)
    cache0 = gen.make_kv_cache(shape, 1, 128, 200, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()

    def plain(n):
        cache, tok = cache0.clone(), tok0.clone()
        pos = torch.tensor([128], dtype=torch.int32, device="cuda")
        logits = torch.empty(1, shape.vocab, device="cuda")
        toks = []
        for _ in range(n):
            dec.kl_decode_step(tok, pos, cache, logits, 1)
            dec.kl_argmax_advance(logits, tok, pos, 1)
            toks.append(int(tok[0]))
        torch.cuda.synchronize()
        return toks, logits.cpu(), cache.cpu().view(torch.uint16)

    ref_toks, ref_logits, ref_cache = plain(5)
    cache, tok = cache0.clone(), tok0.clone()
    pos = torch.tensor([128], dtype=torch.int32, device="cuda")
    logits = torch.empty(1, shape.vocab, device="cuda")
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    toks = []
    with torch.cuda.stream(side):
        dec.kl_decode_step(tok, pos, cache, logits, 1, side)   # first step outside the capture
        dec.kl_argmax_advance(logits, tok, pos, 1, side)
        side.synchronize()
        toks.append(int(tok[0]))
        graph = torch.cuda.CUDAGraph()
        try:
            with torch.cuda.graph(graph, stream=side):
                dec.kl_decode_step(tok, pos, cache, logits, 1, side)
                dec.kl_argmax_advance(logits, tok, pos, 1, side)
        except Exception as exc:
            pytest.skip(f"stream capture of the cooperative launches refused: {exc}")
        for _ in range(4):
            graph.replay()
            side.synchronize()
            toks.append(int(tok[0]))
    assert dec.kl_last_status() == binding.KL_OK
    assert toks == ref_toks
    assert torch.equal(logits.cpu(), ref_logits)
    assert torch.equal(cache.cpu().view(torch.uint16), ref_cache)
    dec.close()


def test_repeated_steps_are_bit_identical():
    """The same step from the same state, several times and in both schedules: identical logits and hidden state.
    Any race between the warps of a CTA or between CTAs (a buffer reused too early) shows up here as run-to-run
    noise long before it breaks the oracle tolerance."""
    import dataclasses
    shape = dataclasses.replace(gen.LLAMA31_8B, n_layers=4)
    context, max_ctx = 4096, 4096 + 8
    dec = helpers.make_decoder(shape, 1, max_ctx, 0)
    cache0 = gen.make_kv_cache(shape, 1, context, max_ctx, 0, "cuda")
    tok = gen.make_tokens(shape, 1, 0).cuda()
    pos = torch.tensor([context], dtype=torch.int32, device="cuda")
    outs = []
    for mode in (binding.KL_MODE_LOOPED,) * 4 + (binding.KL_MODE_PER_LAYER,) * 2 + (binding.KL_MODE_PER_STAGE,) * 2:
        dec.kl_set_mode(mode)
        cache = cache0.clone()
        logits = torch.empty(1, shape.vocab, device="cuda")
        hidden = torch.empty(1, shape.hidden, device="cuda")
        dec.kl_decode_step(tok, pos, cache, logits, 1)
        dec.kl_read_hidden(hidden, 1)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        outs.append((logits.cpu(), hidden.cpu(), cache.cpu().view(torch.uint16)))
    for lg, hd, ch in outs[1:]:
        assert torch.equal(lg, outs[0][0]) and torch.equal(hd, outs[0][1]) and torch.equal(ch, outs[0][2])
    dec.close()


# the bounded waits in both modes of the batch-1 kernels: the tiny shape runs in the plain mode, the other in stash mode
WAIT_SHAPES = {"plain": gen.TINY, "stash": gen.ModelShape(2, 2048, 16, 4, 128, 4096, 1544, 1e-5, 500000.0)}


@pytest.mark.parametrize("mode_name", sorted(WAIT_SHAPES))
def test_bounded_wait_reports_timeout_and_recovers(mode_name):
    """A stage end that is never signalled makes the waits on it run out: the step reports KL_ERR_SYNC_TIMEOUT
    (no hang, no trap) and the next step on the same handle is correct again."""
    shape = WAIT_SHAPES[mode_name]
    dec = helpers.make_decoder(shape, 1, 200, 0)
    assert dec.kl_stash_mode() == (1 if mode_name == "stash" else 0)
    cache = gen.make_kv_cache(shape, 1, 128, 200, 0, "cuda")
    tok = gen.make_tokens(shape, 1, 0).cuda()
    pos = torch.tensor([128], dtype=torch.int32, device="cuda")
    logits_ok = torch.empty(1, shape.vocab, device="cuda")
    logits_bad = torch.empty(1, shape.vocab, device="cuda")
    c1 = cache.clone()
    dec.kl_decode_step(tok, pos, c1, logits_ok, 1)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    dec.kl_set_wait_limit_ns(20_000_000)  # 20 ms
    for stage in (0, 2, 4):
        dec.kl_debug_skip_signal_once(stage)
        dec.kl_decode_step(tok, pos, cache.clone(), logits_bad, 1)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_ERR_SYNC_TIMEOUT
        assert dec.kl_last_status() == binding.KL_OK  # reading clears it
        c2 = cache.clone()
        dec.kl_decode_step(tok, pos, c2, logits_bad, 1)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        assert torch.equal(logits_bad, logits_ok) and torch.equal(c1, c2)
    dec.close()


def test_device_side_range_errors_make_the_step_a_noop():
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 1, 140, 0)
    cache = gen.make_kv_cache(shape, 1, 128, 140, 0, "cuda")
    before = cache.clone()
    logits = torch.full((1, shape.vocab), 7.0, device="cuda")
    for tok, pos in ((shape.vocab, 128), (-1, 128), (3, 140), (3, -2)):
        t = torch.tensor([tok], dtype=torch.int32, device="cuda")
        p = torch.tensor([pos], dtype=torch.int32, device="cuda")
        dec.kl_decode_step(t, p, cache, logits, 1)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_ERR_OUT_OF_RANGE
        assert torch.equal(cache, before) and bool((logits == 7.0).all())
    dec.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 1, 140, 0)
    cache = gen.make_kv_cache(shape, 1, 128, 140, 0, "cuda")
    tok = gen.make_tokens(shape, 1, 0)
    pos = torch.tensor([128], dtype=torch.int32)
    logits_d = torch.empty(1, shape.vocab, device="cuda")
    c1, c2 = cache.clone(), cache.clone()
    dec.kl_decode_step(tok.cuda(), pos.cuda(), c1, logits_d, 1)
    torch.cuda.synchronize()
    logits_h = torch.empty(1, shape.vocab).pin_memory()
    dec.kl_decode_step_host(tok.pin_memory(), pos.pin_memory(), c2, logits_h, 1)
    assert torch.equal(logits_h, logits_d.cpu()) and torch.equal(c1, c2)
    dec.close()


def test_host_buffer_entry_point_batched_graph_replay():
    """kl_decode_step_host keeps a batched step as an instantiated CUDA graph per (cache, batch): the first call
    captures, later calls replay, a different cache or batch captures again.  Every call gives the bits of the
    device-pointer entry point, and a bad token still makes the whole step a no-op that the status word reports."""
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 4, 200, 0)
    cache0 = gen.make_kv_cache(shape, 4, 128, 200, 0, "cuda")
    for batch, caches in ((4, 2), (3, 1)):
        tok = gen.make_tokens(shape, 4, 0)[:batch].contiguous()
        for c in range(caches):
            ref_cache, cache = cache0.clone(), cache0.clone()   # a new tensor: a new cache address
            logits_d = torch.empty(batch, shape.vocab, device="cuda")
            logits_h = torch.empty(batch, shape.vocab).pin_memory()
            for step in range(3):   # capture, replay, replay
                pos = torch.tensor([128, 7, 64, 0][:batch], dtype=torch.int32) + step
                n0 = dec.kl_launch_count()
                dec.kl_decode_step(tok.cuda(), pos.cuda(), ref_cache, logits_d, batch)
                n1 = dec.kl_launch_count()
                dec.kl_decode_step_host(tok.pin_memory(), pos.pin_memory(), cache, logits_h, batch)
                assert dec.kl_launch_count() - n1 == n1 - n0   # a replay counts the kernels it launches
                torch.cuda.synchronize()
                assert dec.kl_last_status() == binding.KL_OK
                assert torch.equal(logits_h, logits_d.cpu()), (batch, c, step)
                assert torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
            bad = tok.clone()
            bad[batch - 1] = shape.vocab + 3
            before = cache.clone()
            logits_h.fill_(7.0)
            dec.kl_decode_step_host(bad.pin_memory(), pos.pin_memory(), cache, logits_h, batch)
            assert dec.kl_last_status() == binding.KL_ERR_OUT_OF_RANGE
            assert torch.equal(cache.view(torch.uint16), before.view(torch.uint16))
    dec.close()


@pytest.mark.parametrize("batch", [1, 4])
def test_greedy_host_entry_point(batch):
    """kl_decode_greedy_host (host tokens and positions in, next tokens out) gives the tokens that kl_decode_step +
    kl_argmax_advance give on device buffers, step after step, for the batch-1 kernels and for the batched path."""
    shape = gen.TINY
    dec = helpers.make_decoder(shape, batch, 200, 0)
    cache0 = gen.make_kv_cache(shape, batch, 128, 200, 0, "cuda")
    tok0 = gen.make_tokens(shape, batch, 0)
    pos0 = torch.tensor([128, 7, 64, 0][:batch], dtype=torch.int32)
    ref_cache, tok_d, pos_d = cache0.clone(), tok0.cuda(), pos0.cuda()
    logits = torch.empty(batch, shape.vocab, device="cuda")
    cache, tok_h, pos_h = cache0.clone(), tok0.clone().pin_memory(), pos0.clone().pin_memory()
    nxt_h = torch.empty(batch, dtype=torch.int32).pin_memory()
    for step in range(4):
        dec.kl_decode_step(tok_d, pos_d, ref_cache, logits, batch)
        dec.kl_argmax_advance(logits, tok_d, pos_d, batch)
        dec.kl_decode_greedy_host(tok_h, pos_h, cache, nxt_h, batch)
        assert dec.kl_last_status() == binding.KL_OK
        assert torch.equal(nxt_h, tok_d.cpu()), step
        tok_h.copy_(nxt_h)
        pos_h.add_(1)
    assert torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
    dec.close()


@pytest.mark.parametrize("name", ["tiny", "odd_rows_hd128", "llama31_8b_4layers"])
def test_one_launch_per_token_matches_four_launches(name):
    """kl_decode_greedy at batch 1 (decoder layers, classifier and sampling in one persistent kernel, the next token's
    embedding prepared by its last CTA) gives, step after step in a chain, the bits of embedding + looped decoder +
    classifier + sampling launched one by one: tokens, positions, logits, final hidden state and cache."""
    import dataclasses
    shape, ctx, steps = {"tiny": (gen.TINY, 128, 8), "odd_rows_hd128": (SHAPES["odd_rows_hd128"], 150, 5),
                         "llama31_8b_4layers": (dataclasses.replace(gen.LLAMA31_8B, n_layers=4), 1024, 4)}[name]
    dec = helpers.make_decoder(shape, 1, ctx + steps + 8, 0)
    cache0 = gen.make_kv_cache(shape, 1, ctx, ctx + steps + 8, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()
    ref_cache, tok, pos = cache0.clone(), tok0.clone(), torch.tensor([ctx], dtype=torch.int32, device="cuda")
    cache, tok1, pos1 = cache0.clone(), tok0.clone(), pos.clone()
    logits, logits1 = torch.empty(1, shape.vocab, device="cuda"), torch.empty(1, shape.vocab, device="cuda")
    hid, hid1 = torch.empty(1, shape.hidden, device="cuda"), torch.empty(1, shape.hidden, device="cuda")
    dec.kl_set_mode(binding.KL_MODE_LOOPED)
    for step in range(steps):
        dec.kl_decode_step(tok, pos, ref_cache, logits, 1)
        dec.kl_read_hidden(hid, 1)
        dec.kl_argmax_advance(logits, tok, pos, 1)
        torch.cuda.synchronize()
        ref = (tok.clone(), pos.clone(), logits.clone(), hid.clone())
        n0 = dec.kl_launch_count()
        # the reference calls in between overwrite the library's activation buffers: the chain restarts every step
        # except where the two runs are kept apart below
        dec.kl_decode_greedy(tok1, pos1, cache, logits1, 1, True)
        assert dec.kl_launch_count() - n0 == 2      # embedding + the one kernel
        dec.kl_read_hidden(hid1, 1)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        assert torch.equal(tok1, ref[0]) and torch.equal(pos1, ref[1]), step
        assert torch.equal(logits1, ref[2]) and torch.equal(hid1, ref[3]), step
    assert torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
    # an uninterrupted chain: one launch per token, the same tokens as the step-by-step run from the same start
    cache2, tok2, pos2 = cache0.clone(), tok0.clone(), torch.tensor([ctx], dtype=torch.int32, device="cuda")
    cache3, tok3, pos3 = cache0.clone(), tok0.clone(), pos2.clone()
    want = []
    for step in range(steps):
        dec.kl_decode_step(tok3, pos3, cache3, logits, 1)
        dec.kl_argmax_advance(logits, tok3, pos3, 1)
        want.append(int(tok3[0]))
    torch.cuda.synchronize()
    got = []
    n0 = dec.kl_launch_count()
    for step in range(steps):
        dec.kl_decode_greedy(tok2, pos2, cache2, logits1, 1, step == 0)
        got.append(tok2.clone())
    torch.cuda.synchronize()
    assert dec.kl_launch_count() - n0 == steps + 1
    assert dec.kl_last_status() == binding.KL_OK
    assert [int(t[0]) for t in got] == want and int(pos2[0]) == ctx + steps
    assert torch.equal(logits1, logits) and torch.equal(cache2.view(torch.uint16), cache3.view(torch.uint16))
    # a call without restart after other decode calls on the handle finds no chain and starts one by itself
    cache4, tok4, pos4 = cache0.clone(), tok0.clone(), torch.tensor([ctx], dtype=torch.int32, device="cuda")
    dec.kl_decode_step(tok3, pos3, cache3, logits, 1)
    dec.kl_decode_greedy(tok4, pos4, cache4, logits1, 1, False)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK and int(tok4[0]) == want[0]
    dec.close()


def test_one_launch_per_token_edge_cases():
    """The chained one-launch step from an empty cache (the first token attends to itself only), on a shape with three
    query heads per kv head and projection biases, against the oracle; and the end of the cache: the step that fills the
    last position succeeds and reports that the next one would not fit, which is then a no-op."""
    import dataclasses
    shape = dataclasses.replace(LLAMA32_3B_2L, qkv_bias=True)
    steps, max_ctx = 3, 16
    host = helpers.HostWeights(shape, 0)
    from oracle import kl_oracle as ko
    orc = ko.Oracle(shape, max_ctx, host.layer, host.globals())
    cache_or = gen.make_kv_cache(shape, 1, 0, max_ctx, 0, "cpu").view(torch.uint16).numpy().copy()
    dec = helpers.make_decoder(shape, 1, max_ctx, 0)
    cache = gen.make_kv_cache(shape, 1, 0, max_ctx, 0, "cuda")
    tok = gen.make_tokens(shape, 1, 0).cuda()
    pos = torch.zeros(1, dtype=torch.int32, device="cuda")
    logits = torch.empty(1, shape.vocab, device="cuda")
    hid = torch.empty(1, shape.hidden, device="cuda")
    t, p = [int(tok[0])], [0]
    for step in range(steps):
        hidden, ref_logits, nxt = orc.step(cache_or, t, p)
        dec.kl_decode_greedy(tok, pos, cache, logits, 1, step == 0)
        dec.kl_read_hidden(hid, 1)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        assert helpers.rel_l2(hid.cpu().numpy()[0], hidden[0]) <= helpers.REL_L2_TOL
        assert helpers.rel_l2(logits.cpu().numpy()[0], ref_logits[0]) <= helpers.REL_L2_TOL
        assert int(tok[0]) == int(nxt[0]) and int(pos[0]) == step + 1
        t, p = [int(nxt[0])], [step + 1]
    # run on to the last position of the cache
    while int(pos[0]) < max_ctx - 1:
        dec.kl_decode_greedy(tok, pos, cache, logits, 1, False)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
    before, tok_before = cache.clone(), tok.clone()
    dec.kl_decode_greedy(tok, pos, cache, logits, 1, False)     # fills position max_ctx - 1
    torch.cuda.synchronize()
    assert int(pos[0]) == max_ctx and not torch.equal(cache.view(torch.uint16), before.view(torch.uint16))
    assert dec.kl_last_status() == binding.KL_ERR_OUT_OF_RANGE   # ... and says that the cache is full
    dec.close()


@pytest.mark.parametrize("name", ["tiny", "odd_rows_hd128", "llama31_8b_4layers", "llama32_3b_2layers_bias", "stash_one_small_layer"])
def test_tokens_per_launch_match_the_chain_of_single_launches(name):
    """kl_decode_greedy_tokens at batch 1 (the loop over layers extended to a loop over tokens: K tokens in one launch)
    gives the bits of K chained one-token launches: picked tokens, final token / position, logits and hidden state of
    the last step, cache.  A second call continues the chain (restart = 0), a one-token launch continues that, and the
    host-buffer entry point returns the same tokens."""
    import dataclasses
    shape, ctx, K = {"tiny": (gen.TINY, 128, 9), "odd_rows_hd128": (SHAPES["odd_rows_hd128"], 150, 5),
                     "llama31_8b_4layers": (dataclasses.replace(gen.LLAMA31_8B, n_layers=4), 1024, 6),
                     "llama32_3b_2layers_bias": (dataclasses.replace(LLAMA32_3B_2L, qkv_bias=True), 0, 7),
                     # stash mode with a whole token's weights on chip at once: producer and stash threads run a token ahead
                     "stash_one_small_layer": (STASH_SHAPES["few_units_rows_of_3072"], 40, 12)}[name]
    total = 2 * K + 1
    dec = helpers.make_decoder(shape, 1, ctx + total + 8, 0)
    cache0 = gen.make_kv_cache(shape, 1, ctx, ctx + total + 8, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()
    pos0 = torch.tensor([ctx], dtype=torch.int32, device="cuda")
    # K + K + 1 chained one-token launches
    ref_cache, tok, pos = cache0.clone(), tok0.clone(), pos0.clone()
    logits, hid = torch.empty(1, shape.vocab, device="cuda"), torch.empty(1, shape.hidden, device="cuda")
    want, want_logits, want_hid = [], [], []
    for step in range(total):
        dec.kl_decode_greedy(tok, pos, ref_cache, logits, 1, step == 0)
        dec.kl_read_hidden(hid, 1)
        want.append(int(tok[0]))
        want_logits.append(logits.clone())
        want_hid.append(hid.clone())
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    # the same as K tokens in one launch, K more in a second one, and a one-token launch behind them
    cache, tok1, pos1 = cache0.clone(), tok0.clone(), pos0.clone()
    logits1, hid1 = torch.empty(1, shape.vocab, device="cuda"), torch.empty(1, shape.hidden, device="cuda")
    out = torch.full((total,), -1, dtype=torch.int32, device="cuda")
    n0 = dec.kl_launch_count()
    dec.kl_decode_greedy_tokens(tok1, pos1, cache, logits1, out, K, 1, True)
    assert dec.kl_launch_count() - n0 == 3            # embedding, the per-token table, the one kernel
    dec.kl_read_hidden(hid1, 1)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    assert out[:K].tolist() == want[:K] and int(tok1[0]) == want[K - 1] and int(pos1[0]) == ctx + K
    assert torch.equal(logits1, want_logits[K - 1]) and torch.equal(hid1, want_hid[K - 1])
    n0 = dec.kl_launch_count()
    dec.kl_decode_greedy_tokens(tok1, pos1, cache, logits1, out[K:], K, 1, False)
    assert dec.kl_launch_count() - n0 == 2            # the chain goes on: no embedding launch
    dec.kl_decode_greedy(tok1, pos1, cache, logits1, 1, False)
    dec.kl_read_hidden(hid1, 1)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    assert out[:2 * K].tolist() == want[:2 * K] and int(tok1[0]) == want[-1] and int(pos1[0]) == ctx + total
    assert torch.equal(logits1, want_logits[-1]) and torch.equal(hid1, want_hid[-1])
    assert torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
    # host buffers
    cache2 = cache0.clone()
    out_h = torch.empty(K, dtype=torch.int32).pin_memory()
    dec.kl_decode_greedy_tokens_host(int(tok0[0]), ctx, cache2, out_h, K)
    assert dec.kl_last_status() == binding.KL_OK
    assert out_h.tolist() == want[:K]
    dec.close()


@pytest.mark.parametrize("name,n_tokens", [("tiny", 700), ("llama31_8b_4layers", 300)])
def test_tokens_per_launch_long_runs(name, n_tokens):
    """Runs longer than one launch holds (256 tokens): the call cuts them into launches that continue one another.  The
    tiny shape is the hard case for the token boundary inside a launch -- a whole token's weight tiles fit into the
    rings, so the copies of a token are requested while the previous token is still being computed and only the wait
    of the producer threads keeps them from reading cache rows that are not written yet."""
    import dataclasses
    shape, ctx = {"tiny": (gen.TINY, 40), "llama31_8b_4layers": (dataclasses.replace(gen.LLAMA31_8B, n_layers=4), 512)}[name]
    dec = helpers.make_decoder(shape, 1, ctx + n_tokens + 8, 0)
    cache0 = gen.make_kv_cache(shape, 1, ctx, ctx + n_tokens + 8, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()
    pos0 = torch.tensor([ctx], dtype=torch.int32, device="cuda")
    ref_cache, tok, pos = cache0.clone(), tok0.clone(), pos0.clone()
    logits = torch.empty(1, shape.vocab, device="cuda")
    want = torch.empty(n_tokens, dtype=torch.int32, device="cuda")
    for step in range(n_tokens):
        dec.kl_decode_greedy(tok, pos, ref_cache, logits, 1, step == 0)
        want[step] = tok[0]
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    for attempt in range(2):
        cache, tok1, pos1 = cache0.clone(), tok0.clone(), pos0.clone()
        logits1 = torch.empty(1, shape.vocab, device="cuda")
        out = torch.full((n_tokens,), -1, dtype=torch.int32, device="cuda")
        n0 = dec.kl_launch_count()
        dec.kl_decode_greedy_tokens(tok1, pos1, cache, logits1, out, n_tokens, 1, True)
        torch.cuda.synchronize()
        assert dec.kl_launch_count() - n0 == 1 + 2 * ((n_tokens + 255) // 256)
        assert dec.kl_last_status() == binding.KL_OK
        assert torch.equal(out, want), (attempt, int((out != want).nonzero()[0]))
        assert int(pos1[0]) == ctx + n_tokens and torch.equal(logits1, logits)
        assert torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
    dec.close()


def test_tokens_per_launch_edge_cases():
    """K tokens per launch against the oracle from an empty cache; a run that would leave the cache is refused on the
    device before anything is decoded; a run that ends exactly at the last position succeeds and reports the full
    cache; batches go through the step-by-step path with the same interface."""
    shape = gen.TINY
    K, max_ctx = 6, 16
    host = helpers.HostWeights(shape, 0)
    from oracle import kl_oracle as ko
    orc = ko.Oracle(shape, max_ctx, host.layer, host.globals())
    cache_or = gen.make_kv_cache(shape, 1, 0, max_ctx, 0, "cpu").view(torch.uint16).numpy().copy()
    dec = helpers.make_decoder(shape, 2, max_ctx, 0)
    cache = gen.make_kv_cache(shape, 1, 0, max_ctx, 0, "cuda")
    tok = gen.make_tokens(shape, 1, 0).cuda()
    pos = torch.zeros(1, dtype=torch.int32, device="cuda")
    logits = torch.empty(1, shape.vocab, device="cuda")
    out = torch.full((max_ctx,), -1, dtype=torch.int32, device="cuda")
    t, p, want = [int(tok[0])], [0], []
    for step in range(K):
        hidden, ref_logits, nxt = orc.step(cache_or, t, p)
        want.append(int(nxt[0]))
        t, p = [int(nxt[0])], [step + 1]
    dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out, K, 1, True)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    assert out[:K].tolist() == want and int(pos[0]) == K
    assert helpers.rel_l2(logits.cpu().numpy()[0], ref_logits[0]) <= helpers.REL_L2_TOL
    # position K, max_ctx - K + 1 more tokens: one too many
    before = cache.clone()
    dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out, max_ctx - K + 1, 1, False)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_ERR_OUT_OF_RANGE
    assert int(pos[0]) == K and torch.equal(cache.view(torch.uint16), before.view(torch.uint16))
    # exactly to the end of the cache
    dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out, max_ctx - K, 1, True)
    torch.cuda.synchronize()
    assert int(pos[0]) == max_ctx
    assert dec.kl_last_status() == binding.KL_ERR_OUT_OF_RANGE   # the cache is full
    # a batch: the same interface, one step after the other
    cache_b0 = gen.make_kv_cache(shape, 2, 5, max_ctx, 1, "cuda")
    tok_b0 = gen.make_tokens(shape, 2, 1).cuda()
    pos_b0 = torch.tensor([5, 2], dtype=torch.int32, device="cuda")
    logits_b = torch.empty(2, shape.vocab, device="cuda")
    ref_cache, tok_b, pos_b, want_b = cache_b0.clone(), tok_b0.clone(), pos_b0.clone(), []
    for _ in range(4):
        dec.kl_decode_greedy(tok_b, pos_b, ref_cache, logits_b, 2, False)
        want_b.append(tok_b.clone())
    cache_b, tok_b, pos_b = cache_b0.clone(), tok_b0.clone(), pos_b0.clone()
    out_b = torch.empty(4, 2, dtype=torch.int32, device="cuda")
    dec.kl_decode_greedy_tokens(tok_b, pos_b, cache_b, logits_b, out_b, 4, 2, True)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    assert torch.equal(out_b, torch.stack(want_b)) and torch.equal(cache_b.view(torch.uint16), ref_cache.view(torch.uint16))
    dec.close()


def test_greedy_chain_of_a_batch_replays_the_cached_graph():
    """kl_decode_greedy for a batch: kl_decode_step + kl_argmax_advance with the step replayed from the graph the handle
    keeps per set of buffers -- same tokens, logits and cache as the two calls made one by one, also after the buffers
    change (a new capture) and inside a caller's own stream capture (no nested replay)."""
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 4, 200, 0)
    cache0 = gen.make_kv_cache(shape, 4, 128, 200, 0, "cuda")
    tok0 = gen.make_tokens(shape, 4, 0).cuda()
    pos0 = torch.tensor([128, 7, 64, 0], dtype=torch.int32, device="cuda")
    ref_cache, tok, pos = cache0.clone(), tok0.clone(), pos0.clone()
    logits = torch.empty(4, shape.vocab, device="cuda")
    want = []
    for _ in range(4):
        dec.kl_decode_step(tok, pos, ref_cache, logits, 4)
        dec.kl_argmax_advance(logits, tok, pos, 4)
        want.append(tok.clone())
    torch.cuda.synchronize()
    for attempt in range(2):   # the second attempt uses new buffers: the graph is captured again
        cache, tok1, pos1, logits1 = cache0.clone(), tok0.clone(), pos0.clone(), torch.empty(4, shape.vocab, device="cuda")
        for step in range(4):
            dec.kl_decode_greedy(tok1, pos1, cache, logits1, 4, step == 0)
            assert torch.equal(tok1, want[step]), (attempt, step)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        assert torch.equal(logits1, logits) and torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
    # inside a caller's capture the step is captured kernel by kernel and replays like any other graph
    cache, tok1, pos1 = cache0.clone(), tok0.clone(), pos0.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            dec.kl_decode_greedy(tok1, pos1, cache, logits1, 4, False, side)
        for step in range(4):
            graph.replay()
        side.synchronize()
    assert torch.equal(tok1, want[3]) and torch.equal(cache.view(torch.uint16), ref_cache.view(torch.uint16))
    dec.close()


@pytest.mark.parametrize("name", ["g4_hd128", "g8_hd64", "g4_hd64"])
def test_cuda_core_attention_loop(name):
    """The CUDA-core attention loop (kl_set_tensor_core_attention(0)) for four and eight query heads per kv head at the
    head sizes that default to the tensor-core loop: all three schedules against the oracle, split-K over several
    chunks with a ragged tail, and -- same arithmetic up to the order of the sums -- close to the tensor-core result."""
    shape = {"g4_hd128": gen.ModelShape(2, 512, 8, 2, 128, 1024, 1000, 1e-5, 500000.0),
             "g8_hd64": gen.ModelShape(2, 512, 8, 1, 64, 768, 1000, 1e-5, 10000.0),
             "g4_hd64": gen.TINY if gen.TINY.n_q_heads // gen.TINY.n_kv_heads == 4 else gen.ModelShape(2, 256, 8, 2, 64, 512, 1024, 1e-5, 10000.0)}[name]
    context, steps, max_ctx = 700, 3, 720
    host = helpers.HostWeights(shape, 4)
    from oracle import kl_oracle as ko
    orc = ko.Oracle(shape, max_ctx, host.layer, host.globals())
    cache0 = gen.make_kv_cache(shape, 1, context, max_ctx, 4, "cuda")
    cache_or = cache0.cpu().view(torch.uint16).numpy().copy()
    dec = helpers.make_decoder(shape, 1, max_ctx, 4)
    results = {}
    for tc in (False, True):
        dec.kl_set_tensor_core_attention(tc)
        for mode in (binding.KL_MODE_LOOPED, binding.KL_MODE_PER_LAYER, binding.KL_MODE_PER_STAGE):
            dec.kl_set_mode(mode)
            cache = cache0.clone()
            logits = torch.empty(1, shape.vocab, device="cuda")
            hidden = torch.empty(1, shape.hidden, device="cuda")
            t, p = gen.make_tokens(shape, 1, 4).tolist(), [context]
            cor = cache_or.copy()
            for s in range(steps):
                ref_hidden, ref_logits, nxt = orc.step(cor, t, p)
                tok_d = torch.tensor(t, dtype=torch.int32, device="cuda")
                pos_d = torch.tensor(p, dtype=torch.int32, device="cuda")
                dec.kl_decode_step(tok_d, pos_d, cache, logits, 1)
                dec.kl_read_hidden(hidden, 1)
                dec.kl_argmax_advance(logits, tok_d, pos_d, 1)
                torch.cuda.synchronize()
                assert dec.kl_last_status() == binding.KL_OK
                lg, hd = logits.cpu().numpy()[0], hidden.cpu().numpy()[0]
                assert helpers.rel_l2(hd, ref_hidden[0]) <= helpers.REL_L2_TOL, (tc, mode, s)
                assert helpers.rel_l2(lg, ref_logits[0]) <= helpers.REL_L2_TOL, (tc, mode, s)
                assert float(np.abs(lg - ref_logits[0]).max()) <= helpers.ABS_LOGIT_TOL, (tc, mode, s)
                assert int(tok_d[0]) == int(nxt[0]), (tc, mode, s)
                t, p = nxt.tolist(), [p[0] + 1]
            results[(tc, mode)] = (logits.cpu(), cache.cpu().view(torch.uint16))
    for tc in (False, True):   # the schedules of one loop agree bit for bit
        for mode in (binding.KL_MODE_PER_LAYER, binding.KL_MODE_PER_STAGE):
            assert torch.equal(results[(tc, mode)][0], results[(tc, binding.KL_MODE_LOOPED)][0])
            assert torch.equal(results[(tc, mode)][1], results[(tc, binding.KL_MODE_LOOPED)][1])
    dec.close()


def test_two_handles_of_different_shapes_step_alternately():
    """Two models alive at once (a small one and one with hidden 8192, whose persistent kernels need different amounts of
    shared memory): creating the second must not take shared memory away from the first.  Both step alternately, on
    every schedule, and give the bits each gives alone."""
    small, wide = gen.TINY, SHAPES["wide_hidden_g8"]

    def run(dec, shape, n):
        cache = gen.make_kv_cache(shape, 1, 100, 120, 0, "cuda")
        tok = gen.make_tokens(shape, 1, 0).cuda()
        pos = torch.tensor([100], dtype=torch.int32, device="cuda")
        logits = torch.empty(1, shape.vocab, device="cuda")
        outs = []
        for i in range(n):
            dec.kl_set_mode(i % 3)
            dec.kl_decode_step(tok, pos, cache, logits, 1)
            dec.kl_argmax_advance(logits, tok, pos, 1)
            outs.append(logits.clone())
            yield
        dec.kl_decode_greedy(tok, pos, cache, logits, 1, True)
        outs.append(logits.clone())
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        run.results[shape.hidden] = outs
        yield

    def alone(shape):
        dec = helpers.make_decoder(shape, 1, 120, 0)
        run.results = {}
        for _ in run(dec, shape, 3):
            pass
        dec.close()
        return run.results[shape.hidden]

    want_small, want_wide = alone(small), alone(wide)
    a = helpers.make_decoder(wide, 1, 120, 0)      # the larger shared-memory request first, then the smaller one
    b = helpers.make_decoder(small, 1, 120, 0)
    run.results = {}
    for _ in zip(run(a, wide, 3), run(b, small, 3)):
        pass
    for got, want in ((run.results[wide.hidden], want_wide), (run.results[small.hidden], want_small)):
        assert len(got) == len(want) and all(torch.equal(g, w) for g, w in zip(got, want))
    a.close()
    b.close()


@pytest.mark.parametrize("mode_name", sorted(WAIT_SHAPES))
def test_bounded_wait_on_the_greedy_chain_leaves_token_and_position_alone(mode_name):
    """A wait that runs out inside the one-launch-per-token kernel: the call reports KL_ERR_SYNC_TIMEOUT, does not touch
    the token or the position (the step's logits and cache row are undefined), and the next call starts a new chain that
    gives the bits of an undisturbed run."""
    shape = WAIT_SHAPES[mode_name]
    dec = helpers.make_decoder(shape, 1, 200, 0)
    assert dec.kl_stash_mode() == (1 if mode_name == "stash" else 0)
    cache0 = gen.make_kv_cache(shape, 1, 128, 200, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()
    logits_ok, logits = torch.empty(1, shape.vocab, device="cuda"), torch.empty(1, shape.vocab, device="cuda")
    c1, tok, pos = cache0.clone(), tok0.clone(), torch.tensor([128], dtype=torch.int32, device="cuda")
    dec.kl_decode_greedy(tok, pos, c1, logits_ok, 1, True)
    torch.cuda.synchronize()
    assert dec.kl_last_status() == binding.KL_OK
    want_tok = int(tok[0])
    dec.kl_set_wait_limit_ns(20_000_000)   # 20 ms
    for stage in (0, 1, 3):
        c2, tok, pos = cache0.clone(), tok0.clone(), torch.tensor([128], dtype=torch.int32, device="cuda")
        dec.kl_debug_skip_signal_once(stage)
        dec.kl_decode_greedy(tok, pos, c2, logits, 1, True)
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_ERR_SYNC_TIMEOUT
        assert int(tok[0]) == int(tok0[0]) and int(pos[0]) == 128
        c2 = cache0.clone()
        dec.kl_decode_greedy(tok, pos, c2, logits, 1, False)    # no restart asked for: the handle starts a chain by itself
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        assert int(tok[0]) == want_tok and int(pos[0]) == 129
        assert torch.equal(logits, logits_ok) and torch.equal(c1.view(torch.uint16), c2.view(torch.uint16))
    dec.close()


def test_step_numbers_wrap_without_a_stale_tag():
    """The step numbers behind the tags wrap after about 2^28 / n_layers steps: the tagged scratch areas are cleared at
    that launch boundary and the numbering restarts.  With the counter preset just below the wrap, a run that crosses
    it -- step by step, as a greedy chain, and as one multi-token launch -- gives the bits of a run far from it."""
    shape = gen.TINY
    dec = helpers.make_decoder(shape, 1, 200, 0)
    wrap = dec.kl_debug_set_step()
    assert wrap == (1 << 28) // shape.n_layers - 260
    cache0 = gen.make_kv_cache(shape, 1, 128, 200, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()
    n = 12

    def chain(kind):
        cache, tok, pos = cache0.clone(), tok0.clone(), torch.tensor([128], dtype=torch.int32, device="cuda")
        logits = torch.empty(1, shape.vocab, device="cuda")
        out = torch.empty(n, dtype=torch.int32, device="cuda")
        if kind == "tokens":
            dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out[:5], 5, 1, True)
            dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out[5:], n - 5, 1, False)
        else:
            for i in range(n):
                if kind == "steps":
                    dec.kl_decode_step(tok, pos, cache, logits, 1)
                    dec.kl_argmax_advance(logits, tok, pos, 1)
                else:
                    dec.kl_decode_greedy(tok, pos, cache, logits, 1, i == 0)
                out[i] = tok[0]
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        return out.cpu(), logits.cpu(), cache.cpu().view(torch.uint16)

    want = chain("steps")
    for kind in ("steps", "greedy", "tokens"):
        for start in (wrap - 4, wrap - 1, wrap - 7):
            dec.kl_debug_set_step(start)
            got = chain(kind)
            assert all(torch.equal(g, w) for g, w in zip(got, want)), (kind, start)
    dec.close()


@pytest.mark.parametrize("name,steps", [("tiny", 1500), ("llama31_8b_4layers", 150), ("stash_one_small_layer", 800)])
def test_sync_protocol_under_seeded_jitter(name, steps):
    """Stress of the exchanges that replace kernel boundaries (tagged words, the gate/up counter, the token boundary
    inside a launch): with kl_debug_set_jitter every CTA sleeps a seeded pseudo-random time of up to 20 us whenever it
    enters a stage, so the CTAs reach every exchange in a different order on every step.  A long greedy run on the
    looped kernel, on the one-launch-per-token chain and as multi-token launches must pick, token for token, what the
    undisturbed per-layer schedule picks, and leave the same cache; no bounded wait may run out."""
    import dataclasses
    shape, ctx = {"tiny": (gen.TINY, 40), "llama31_8b_4layers": (dataclasses.replace(gen.LLAMA31_8B, n_layers=4), 512),
                  # stash mode, a whole token's weights on chip at once: the stash threads run a token ahead of the consumers
                  "stash_one_small_layer": (STASH_SHAPES["few_units_rows_of_3072"], 40)}[name]
    dec = helpers.make_decoder(shape, 1, ctx + steps + 8, 0)
    cache0 = gen.make_kv_cache(shape, 1, ctx, ctx + steps + 8, 0, "cuda")
    tok0 = gen.make_tokens(shape, 1, 0).cuda()

    def run(kind):
        cache, tok = cache0.clone(), tok0.clone()
        pos = torch.tensor([ctx], dtype=torch.int32, device="cuda")
        logits = torch.empty(1, shape.vocab, device="cuda")
        out = torch.empty(steps, dtype=torch.int32, device="cuda")
        if kind == "tokens":
            dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out, steps, 1, True)
        else:
            for i in range(steps):
                if kind == "greedy":
                    dec.kl_decode_greedy(tok, pos, cache, logits, 1, i == 0)
                else:
                    dec.kl_decode_step(tok, pos, cache, logits, 1)
                    dec.kl_argmax_advance(logits, tok, pos, 1)
                out[i] = tok[0]
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK, kind
        return out.cpu(), logits.cpu(), cache.cpu().view(torch.uint16)

    dec.kl_set_mode(binding.KL_MODE_PER_LAYER)
    want = run("steps")
    dec.kl_set_mode(binding.KL_MODE_LOOPED)
    for seed, kind in ((1, "steps"), (2, "greedy"), (3, "tokens"), (4, "tokens")):
        dec.kl_debug_set_jitter(seed, 20_000)
        got = run(kind)
        first_diff = int((got[0] != want[0]).nonzero()[0]) if not torch.equal(got[0], want[0]) else -1
        assert first_diff < 0, (kind, seed, first_diff)
        assert torch.equal(got[1], want[1]) and torch.equal(got[2], want[2]), (kind, seed)
    dec.kl_debug_set_jitter(0, 0)
    dec.close()


MOE_SHAPES = {
    # the tiny decoder with four experts, two per token
    "tiny_4x2": gen.ModelShape(4, 256, 4, 2, 64, 512, 1024, 1e-5, 10000.0, False, 4, 2),
    # eight experts, two per token, FFN wider than a ring slot (the down projection in column pieces per expert), G = 4, head size 128
    "hd128_8x2_split_down": gen.ModelShape(2, 512, 8, 2, 128, 3072, 1000, 1e-5, 500000.0, False, 8, 2),
    # one expert per token, three experts, row counts that are no multiples of the CTA count
    "odd_3x1": gen.ModelShape(3, 328, 8, 2, 128, 1008, 1544, 1e-5, 500000.0, False, 3, 1),
}


@pytest.mark.parametrize("name", sorted(MOE_SHAPES))
def test_mixture_of_experts_decoder(name):
    """Decoders whose MLP is a mixture of experts (the paper's Table 2 lists one): router, top-k, gate weights and the
    gathered expert MLPs run inside the looped kernel -- the expert tiles are the one part of the weight stream whose
    addresses depend on an activation.  All three schedules against the oracle for several steps (the router must pick
    the oracle's experts or the logits would be far off), bit-identical to each other; then the one-launch-per-token
    chain and a multi-token launch pick the same tokens; a batch decodes sequence after sequence."""
    shape = MOE_SHAPES[name]
    rep = helpers.run_parity(shape, context=150, steps=6, seed=2)
    helpers.assert_parity(rep, 6)
    want = [r["next"][0] for r in rep["ref"]]
    dec = helpers.make_decoder(shape, 1, 170, 2)
    for kind in ("greedy", "tokens"):
        cache = gen.make_kv_cache(shape, 1, 150, 170, 2, "cuda")
        tok = gen.make_tokens(shape, 1, 2).cuda()
        pos = torch.tensor([150], dtype=torch.int32, device="cuda")
        logits = torch.empty(1, shape.vocab, device="cuda")
        out = torch.empty(6, dtype=torch.int32, device="cuda")
        if kind == "tokens":
            dec.kl_decode_greedy_tokens(tok, pos, cache, logits, out, 6, 1, True)
        else:
            for i in range(6):
                dec.kl_decode_greedy(tok, pos, cache, logits, 1, i == 0)
                out[i] = tok[0]
        torch.cuda.synchronize()
        assert dec.kl_last_status() == binding.KL_OK
        assert out.tolist() == want, kind
    dec.close()
    rep = helpers.run_parity(shape, context=150, steps=2, seed=2, batch=3, positions0=[5, 64, 150], modes=(binding.KL_MODE_LOOPED,))
    helpers.assert_parity(rep, 2, batch=3)


def test_mixtral_8x7b_shape_two_layers():
    """The mixture-of-experts decoder of the paper's Table 2 by its public dimensions (hidden 4096, 32 / 8 heads of 128,
    8 experts of FFN 14336 with 2 per token: per expert the down projection in ten column pieces, twenty per row unit),
    two layers, context 1024, three steps, all schedules."""
    shape = gen.ModelShape(2, 4096, 32, 8, 128, 14336, 32000, 1e-5, 1000000.0, False, 8, 2)
    rep = helpers.run_parity(shape, context=1024, steps=3, seed=0, max_ctx=1024 + 8, check_cache=False)
    helpers.assert_parity(rep, 3, check_cache=False)
