"""Parity at FULL depth for the large configurations: every layer of the model through the C ABI against the
layer-streaming oracle, two teacher-forced decode steps each (the sampled-layer tests of test_parity_gpu.py cover the
same shapes with more steps and more positions, on two layers).  Tolerances as everywhere: rel-L2 <= 1e-2 on hidden
state and logits, max |delta logit| <= 5e-2, identical greedy tokens."""
import pytest

from paper_2410_23668_b200 import inputs as gen
from tests import helpers

pytestmark = pytest.mark.gpu


def test_llama31_8b_context_65536_all_layers():
    """Config 3: the 8B shape, batch 1, 65536 cached positions (8.6 GB of cache), all 32 layers: every split-K unit
    streams ~3640 positions per layer."""
    worst = helpers.run_full_depth(gen.LLAMA31_8B, context=65536, steps=2)
    print("config 3, 32 layers:", worst)


def test_llama31_8b_context_65536_all_layers_one_launch_per_token():
    """The same configuration on the one-launch-per-token schedule (decoder layers, classifier and sampling in one
    persistent kernel)."""
    worst = helpers.run_full_depth(gen.LLAMA31_8B, context=65536, steps=2, greedy_chain=True)
    print("config 3, one launch per token:", worst)


def test_llama31_8b_batch_32_context_4096_all_layers():
    """Config 4: the 8B shape, 32 sequences of 4096 cached positions each (17 GB of cache), all 32 layers on the batched
    tensor-core path.  The oracle decodes sequences 0, 13 and 31 (sequences are independent); the other 29 are checked
    for finite results."""
    worst = helpers.run_full_depth(gen.LLAMA31_8B, context=4096, steps=2, batch=32, oracle_rows=[0, 13, 31], batched_path=True)
    print("config 4, 32 layers:", worst)


def test_llama31_70b_all_layers():
    """Config 5: the 70B shape (80 layers, hidden 8192, FFN 28672; 139 GB of weights generated layer by layer on the
    device and, for the oracle, layer by layer on the host), batch 1, context 4096."""
    worst = helpers.run_full_depth(gen.LLAMA31_70B, context=4096, steps=2)
    print("config 5, 80 layers:", worst)


def test_mixtral_8x7b_shape_all_layers():
    """The mixture-of-experts decoder at full depth: 32 layers of 8 experts (93 GB of weights on the device, one layer at
    a time on the host), batch 1, context 4096; 64 routing decisions per step have to agree with the oracle's."""
    shape = gen.ModelShape(32, 4096, 32, 8, 128, 14336, 32000, 1e-5, 1000000.0, False, 8, 2)
    worst = helpers.run_full_depth(shape, context=4096, steps=2)
    print("mixture of experts, 32 layers:", worst)
