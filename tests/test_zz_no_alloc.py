"""GPU test of kl_argmax_advance_static: the sampling block whose scratch is a fixed array inside the library.

The file name sorts last so that the test also runs after every other GPU test has used the device; it passes on
its own as well.  The expected values come from the existing entry point kl_argmax_advance (integer results:
compared exactly) and from torch.argmax on the same logits.
"""
import pytest
import torch

from paper_2410_23668_b200 import binding, inputs as gen

pytestmark = pytest.mark.gpu


def _logits(batch: int, vocab: int, seed: int) -> torch.Tensor:
    g = torch.Generator().manual_seed(seed)
    x = torch.randn(batch, vocab, generator=g)
    # ties: the maximum appears several times in some rows, the lowest index has to win
    for b in range(0, batch, 2):
        hi = x[b].max() + 1.0
        idx = torch.randint(0, vocab, (3,), generator=g)
        x[b, idx] = hi
    return x.cuda()


def _first_max(logits: torch.Tensor) -> torch.Tensor:
    """Lowest index among the maxima of every row."""
    mx = logits.max(dim=1, keepdim=True).values
    ar = torch.arange(logits.shape[1], device=logits.device).expand_as(logits)
    big = torch.full_like(ar, logits.shape[1])
    return torch.where(logits == mx, ar, big).min(dim=1).values.to(torch.int32)


def test_static_argmax_matches_handle_entry_point_twice():
    shape = gen.TINY
    batch = 5
    dec = binding.Decoder(shape, max_batch=batch, max_ctx=64)
    try:
        for call in range(2):  # two calls in a row share the array: the second must not see the first one's state
            logits = _logits(batch, shape.vocab, seed=100 + call)
            start = torch.arange(10, 10 + batch, dtype=torch.int32, device="cuda")
            tok_ref = torch.full((batch,), -1, dtype=torch.int32, device="cuda")
            pos_ref = start.clone()
            dec.kl_argmax_advance(logits, tok_ref, pos_ref, batch)
            tok = torch.full((batch,), -1, dtype=torch.int32, device="cuda")
            pos = start.clone()
            binding.kl_argmax_advance_static(logits, tok, pos, batch)
            torch.cuda.synchronize()
            assert torch.equal(tok, tok_ref)
            assert torch.equal(pos, pos_ref)
            assert torch.equal(pos, start + 1)
            assert torch.equal(tok, _first_max(logits))
    finally:
        dec.close()


def test_static_argmax_full_vocab_and_side_stream():
    vocab, batch = 128256, 3
    logits = _logits(batch, vocab, seed=7)
    st = torch.cuda.Stream()
    st.wait_stream(torch.cuda.current_stream())
    tok = torch.zeros(batch, dtype=torch.int32, device="cuda")
    pos = torch.zeros(batch, dtype=torch.int32, device="cuda")
    with torch.cuda.stream(st):
        binding.kl_argmax_advance_static(logits, tok, pos, batch, stream=st)
    st.synchronize()
    assert torch.equal(tok, _first_max(logits))
    assert torch.equal(pos, torch.ones(batch, dtype=torch.int32, device="cuda"))


def test_static_argmax_at_the_maximum_batch():
    batch, vocab = binding.KL_STATIC_ARGMAX_MAX_BATCH, 1003   # ragged: 1003 is not a multiple of the block count
    logits = _logits(batch, vocab, seed=11)
    tok = torch.zeros(batch, dtype=torch.int32, device="cuda")
    pos = torch.full((batch,), 41, dtype=torch.int32, device="cuda")
    for _ in range(2):
        binding.kl_argmax_advance_static(logits, tok, pos, batch)
    torch.cuda.synchronize()
    assert torch.equal(tok, _first_max(logits))
    assert int((pos != 43).sum()) == 0


def test_static_argmax_rejects_sizes_beyond_the_array():
    too_many = binding.KL_STATIC_ARGMAX_MAX_BATCH + 1
    logits = torch.zeros(too_many, 8, device="cuda")
    tok = torch.full((too_many,), -7, dtype=torch.int32, device="cuda")
    pos = torch.zeros(too_many, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.KlError) as e:
        binding.kl_argmax_advance_static(logits, tok, pos, too_many)
    assert e.value.code == binding.KL_ERR_TOO_LARGE
    assert "KL_ERR_TOO_LARGE" in str(e.value)
    torch.cuda.synchronize()
    assert int((tok != -7).sum()) == 0 and int(pos.sum()) == 0  # nothing was launched


def test_static_argmax_allocates_no_device_memory():
    """What the entry point is for: after its first call on the device (which looks up the array's address), a call
    leaves the amount of free device memory exactly where it was -- nothing is allocated, by the library or inside the
    CUDA runtime on its behalf.  All buffers of the test exist before the measurement starts."""
    batch, vocab = 4, 4099
    logits = _logits(batch, vocab, seed=3)
    tok = torch.zeros(batch, dtype=torch.int32, device="cuda")
    pos = torch.zeros(batch, dtype=torch.int32, device="cuda")
    binding.kl_argmax_advance_static(logits, tok, pos, batch)   # the first call on this device may set up
    torch.cuda.synchronize()
    free0, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        binding.kl_argmax_advance_static(logits, tok, pos, batch)
    torch.cuda.synchronize()
    free1, _ = torch.cuda.mem_get_info()
    assert free1 == free0
    assert torch.equal(tok, _first_max(logits)) and int((pos != 4).sum()) == 0
