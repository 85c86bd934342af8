"""GPU tests of the library's microbenchmarks: they run, and what they report is physically plausible for a
B200 (the figures themselves are reported by bench.py, not asserted tightly here)."""
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


def test_fadd_peak_is_near_the_derived_rate(som_mod):
    """SMs x 128 lanes x clock: the measured add rate lies within 80 .. 101 % of it at the maximum clock."""
    props = torch.cuda.get_device_properties(0)
    derived = props.multi_processor_count * 128 * 1.965e9
    got = som_mod.measure_fadd_peak()
    assert 0.5 * derived < got < 1.01 * derived * (2100.0 / 1965.0)


def test_operand_paths(som_mod):
    """Shared memory delivers at most 128 bytes per clock and SM and close to it on conflict-free rows; rows
    from L2 come slower than from shared memory, by either route; two streams together move more bytes per
    clock than the L2 stream alone."""
    p = som_mod.measure_operand_paths()
    assert 90.0 < p["shared"] <= 128.5
    assert 20.0 < p["l2_global"] < p["shared"]
    assert 20.0 < p["l2_texture"] < p["shared"]
    assert p["shared_and_l2"] > p["l2_global"]
