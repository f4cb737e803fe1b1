"""GPU parity of the redundancy analysis map (mixkv_similarity_map) against the plain pairwise
definition in oracle/similarity_plain.py."""
import numpy as np
import pytest
import torch

from oracle import similarity_plain
from paper_2510_20707_b200 import binding, synth

pytestmark = pytest.mark.gpu
ATOL, RTOL = 2e-5, 2e-4   # fp32 sums of up to `block` unit rows and 128-term dot products


def run(X_bits, block):
    X = torch.from_numpy(X_bits.view(np.int16)).cuda().view(torch.bfloat16)
    cells, mean = binding.similarity_map(X, block)
    torch.cuda.synchronize()
    ref_cells, ref_mean = similarity_plain.block_cosine_map(X_bits, block)
    assert np.allclose(cells.cpu().numpy(), ref_cells, rtol=RTOL, atol=ATOL)
    assert np.allclose(mean.cpu().numpy(), ref_mean, rtol=RTOL, atol=ATOL)
    return cells, mean


@pytest.mark.parametrize("H,L,block", [(3, 1000, 64), (2, 40, 1), (1, 1, 8), (2, 129, 128),
                                       (4, 777, 100), (2, 3000, 700)])
def test_random_rows_with_shared_component(H, L, block):
    rng = np.random.default_rng(L)
    X = rng.standard_normal((H, L, 128)) + 1.3 * rng.standard_normal((H, 1, 128))
    if L > 10:
        X[0, 5] = 0.0                       # a zero row has cosine 0 with everything
    run(synth.f32_to_bf16_bits(X.astype(np.float32)), block)


def test_keys_and_values_of_a_c2_layer():
    wl = synth.CONFIGS["C2"]
    x = synth.make_layer(wl, 7, "calibrated")
    cells, mean = run(x["K"], 128)
    # vision keys are built around shared centroids and a shared offset: redundant, as in the paper
    assert float(mean.min()) > 0.2
    run(x["V"], 256)


def test_rejects_bad_arguments():
    X = torch.zeros((1, 16, 64), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(binding.MixKVError):
        binding.similarity_map(X, 4)        # head_dim must be 128
