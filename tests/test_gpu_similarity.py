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


@pytest.mark.parametrize("H,L,block", [(2, 1000, 16), (1, 700, 4), (3, 300, 2), (2, 257, 1),
                                       (1, 130, 8), (2, 2049, 16), (1, 128, 1), (2, 391, 4)])
def test_dense_route_small_maps(H, L, block):
    # block = 1, 2, 4, 8, 16 takes the tensor-core route: ragged last tile and last block, a zero
    # row, diagonal cells without the i == j pairs
    rng = np.random.default_rng(1000 * block + L)
    X = rng.standard_normal((H, L, 128)) + 0.8 * rng.standard_normal((H, 1, 128))
    X[0, 3] = 0.0
    cells, _ = run(synth.f32_to_bf16_bits(X.astype(np.float32)), block)
    c = cells.cpu().numpy()
    # mirrored tiles are the same numbers; inside a diagonal tile (i, j) and (j, i) are summed in
    # a different order
    assert np.allclose(c, c.transpose(0, 2, 1), rtol=0, atol=1e-6)
    if block == 1:
        assert (np.diagonal(c, axis1=1, axis2=2) == 0).all()


@pytest.mark.parametrize("L,block", [(8192, 1), (32768, 16)])
def test_dense_route_full_size_sampled(L, block):
    # The dense map of the keys of two heads at full size.  The pairwise oracle needs the L x L
    # matrix in fp64, so it checks sampled 128-row tiles: a cell depends only on the rows of its
    # two blocks, and the oracle run on the rows of tiles a and b gives the cells of (a, a),
    # (a, b), (b, a), (b, b).  The whole map is checked for symmetry and range, its mean against
    # Eq. 4 from the oracle's key geometry.
    import oracle
    wl = synth.replace(synth.CONFIGS["C3"], seq_lens=(L,), vision_tokens=(L - 256,),
                       frame_tokens=(L - 256) // 32)
    K = synth.make_layer(wl, 3, "calibrated")["K"][:2]
    X = torch.from_numpy(K.view(np.int16)).cuda().view(torch.bfloat16)
    cells, mean = binding.similarity_map(X, block)
    torch.cuda.synchronize()
    nT, per = L // 128, 128 // block
    for h in range(2):
        for a, b in ((0, 1), (5, nT - 1), (nT // 2, nT // 2 + 7), (nT - 2, nT - 1)):
            rows = np.concatenate([np.arange(a * 128, a * 128 + 128), np.arange(b * 128, b * 128 + 128)])
            ref, _ = similarity_plain.block_cosine_map(K[h:h + 1, rows], block)
            ia, ib = slice(a * per, a * per + per), slice(b * per, b * per + per)
            got = torch.cat([torch.cat([cells[h, ia, ia], cells[h, ia, ib]], 1),
                             torch.cat([cells[h, ib, ia], cells[h, ib, ib]], 1)], 0).cpu().numpy()
            assert np.allclose(got, ref[0], rtol=RTOL, atol=ATOL), (h, a, b)
        assert torch.allclose(cells[h], cells[h].T, rtol=0, atol=1e-6)
        assert float(cells[h].abs().max()) <= 1.0 + 1e-4
    rbar = np.array([oracle.key_geometry(K[h])[1] for h in range(2)])
    assert np.allclose(mean.cpu().numpy(), rbar, rtol=RTOL, atol=ATOL)


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
