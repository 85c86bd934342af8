"""The tcgen05 probe (densified hot-feature tile): its tensor-core partial scores must be the plain sums
they stand for.  Reference: h_n - sum over the sample's dense features of w[f, n], written out in fp64
with numpy from the same inputs (the definition of the gather-sum, Section 3.3 / Eq. 1)."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def som_mod():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_24067_b200 import som
    som.load_library()
    return som


def _inputs(H, n_tiles, seed, density):
    rng = np.random.default_rng(seed)
    rows = rng.random((H, 64)).astype(np.float32)
    rows[rng.random((H, 64)) < 0.8] *= 0.05          # mostly small weights with a few large ones
    hnorm = (10.0 + 10.0 * rng.random(64)).astype(np.float32)
    member = rng.random((n_tiles * 128, H)) < density
    member[0, :] = True                               # one sample with every dense feature
    member[1, :] = False                              # and one with none
    words = np.zeros((n_tiles * 128, H // 32), np.uint32)
    for f in range(H):
        words[:, f // 32] |= member[:, f].astype(np.uint32) << np.uint32(f % 32)
    return rows, hnorm, member, words


@pytest.mark.parametrize("H,terms", [(32, 2), (64, 1), (64, 2), (128, 2), (256, 1), (256, 2)])
def test_partial_scores_of_the_first_tile(som_mod, H, terms):
    n_tiles = 3
    rows, hnorm, member, words = _inputs(H, n_tiles, 7 + H + terms, 0.08)
    r = som_mod.tc_probe(torch.from_numpy(rows).cuda(), torch.from_numpy(hnorm).cuda(),
                         torch.from_numpy(words.view(np.int32)).cuda(), H, terms, n_tiles, mode=7, repeats=2,
                         blocks=2)
    torch.cuda.synchronize()
    assert int(r["status"].item()) == 0, "a bounded wait inside the probe gave up"
    want = hnorm.astype(np.float64)[None, :] - member[:128].astype(np.float64) @ rows.astype(np.float64)
    got = r["out"].cpu().numpy().astype(np.float64)
    err = np.abs(got - want).max()
    # two fp16 terms carry 22 bits of every weight and three of the seed; one term rounds every weight
    # to fp16 (2^-11 relative).  fp32 accumulation of up to H + 3 products on top.
    tol = 2e-4 if terms == 2 else H * 2.5e-4
    assert err <= tol, (H, terms, err)
    # last tile walked: tile (2 * n_tiles - 1) % n_tiles, minimum over the 64 neurons per sample
    last = (2 * n_tiles - 1) % n_tiles
    want_min = (hnorm.astype(np.float64)[None, :] -
                member[last * 128:(last + 1) * 128].astype(np.float64) @ rows.astype(np.float64)).min(axis=1)
    for b in range(2):
        assert np.abs(r["mins"][b].cpu().numpy() - want_min).max() <= tol
    assert (r["cycles"].cpu().numpy() > 0).all()
