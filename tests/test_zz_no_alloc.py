"""som_norms_noalloc, the entry point for callers that cannot allocate device memory
(their memory belongs to a pool of their own, or they cannot take the synchronisation an
allocation may imply): it must give the same norms as the handle-based som_norms, and both must
be the CPU oracle's fp64 norms rounded to fp32.

Collected last on purpose, so that a run stopping at the first failure has already run every
other test; it passes alone in a fresh process as well as after the others.
"""
import numpy as np
import pytest
import torch

from oracle import som_oracle as orc
from paper_2608_24067_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()
    return som


def _reference_norms(som_mod, V, M, W):
    h = som_mod.Som(V, M, W)
    h.norms()
    out = h.get_norms()
    torch.cuda.synchronize()
    return out


def test_noalloc_norms_match_handle_norms_twice_in_a_row(som_mod):
    # two different codebooks and shapes back to back: the shared scratch keeps the first
    # call's contents, the second call must not see them
    shapes = [(2000, 256, 0), (3000, 4096, 1)]
    outs = []
    for V, M, seed in shapes:
        W = synth.fill_codebook(V, M, seed, device="cuda")
        out = torch.full((M,), -1.0, dtype=torch.float32, device="cuda")
        som_mod.norms_noalloc(V, M, W, out)
        outs.append((V, M, W, out))
    torch.cuda.synchronize()
    for V, M, W, out in outs:
        ref = _reference_norms(som_mod, V, M, W)
        # same fp64 accumulation, possibly split differently over V: one fp32 rounding apart at most
        np.testing.assert_allclose(out.cpu().numpy(), ref.cpu().numpy(), rtol=2e-7, atol=0.0)
        # and against the oracle: ascending-v fp64 sums of squares, one fp32 rounding on the GPU side
        want = orc.norms(W.cpu().numpy(), V, M)
        np.testing.assert_allclose(out.cpu().numpy().astype(np.float64), want, rtol=2e-7, atol=0.0)
    # the same call again gives bit-identical output (fixed summation order)
    V, M, W, out = outs[1]
    again = torch.empty_like(out)
    som_mod.norms_noalloc(V, M, W, again)
    torch.cuda.synchronize()
    assert torch.equal(again, out)


def test_noalloc_unaligned_neuron_count(som_mod):
    V, M = 257, 130  # M % 4 != 0: scalar path
    W = torch.rand(V * M, device="cuda")
    out = torch.empty(M, dtype=torch.float32, device="cuda")
    som_mod.norms_noalloc(V, M, W, out)
    ref = _reference_norms(som_mod, V, M, W)
    np.testing.assert_allclose(out.cpu().numpy(), ref.cpu().numpy(), rtol=2e-7, atol=0.0)
    want = orc.norms(W.cpu().numpy(), V, M)
    np.testing.assert_allclose(out.cpu().numpy().astype(np.float64), want, rtol=2e-7, atol=0.0)


def test_noalloc_rejects_sizes_beyond_its_scratch(som_mod):
    M = som_mod.NOALLOC_MAX_M + 4
    W = torch.zeros(2 * M, device="cuda")
    out = torch.empty(M, dtype=torch.float32, device="cuda")
    with pytest.raises(som_mod.SomError) as e:
        som_mod.norms_noalloc(2, M, W, out)
    assert e.value.status == 3  # SOM_ERR_UNSUPPORTED
