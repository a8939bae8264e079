"""granq_range_noalloc(): the range entry point for callers that cannot allocate device memory
(allocator callbacks, plugins that only get their buffers, loops that must avoid the driver's
allocator).  Its scratch is an array inside the library, shared by all calls, so the check is
that it gives exactly what granq_range() gives with a caller workspace - on two calls in a row,
the second on different data with fewer groups, so stale keys from the first call would show."""
import numpy as np
import pytest
import torch

from oracle import granq_oracle as orc

pytestmark = pytest.mark.gpu


def _bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy().view(np.uint32)


def _oracle_range(x: torch.Tensor, group: int):
    """Eq. 4 by the CPU oracle on the same values (bf16 tensors go in as their bit patterns)."""
    if x.dtype == torch.bfloat16:
        return orc.range_(x.view(torch.int16).cpu().numpy().view(np.uint16), group_mode=group)
    return orc.range_(x.cpu().numpy(), group_mode=group)


@pytest.fixture(scope="module")
def b():
    from paper_2503_18339_b200 import binding
    binding.lib()
    return binding


def _pair(b, x, group):
    lo_ref, hi_ref = b.granq_range(x, group=group)
    G = b.num_groups(x.shape, 1, group)
    lo = torch.full((G,), float("nan"), device="cuda")
    hi = torch.full((G,), float("nan"), device="cuda")
    b.granq_range_noalloc(x, lo, hi, group=group)
    torch.cuda.synchronize()
    return lo, hi, lo_ref, hi_ref


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_two_calls_in_a_row_match_the_workspace_entry_point(b, dtype):
    g = torch.Generator(device="cuda").manual_seed(5)
    first = (torch.randn(6, 40, 14, 14, device="cuda", generator=g) * 3 + 1).to(dtype)
    second = (torch.randn(3, 8, 7, 7, device="cuda", generator=g) * 0.01).to(dtype)   # smaller range, fewer groups
    for x, group in ((first, b.GROUP_SAMPLE_CHANNEL), (second, b.GROUP_CHANNEL), (first, b.GROUP_TENSOR)):
        lo, hi, lo_ref, hi_ref = _pair(b, x, group)
        assert torch.equal(lo, lo_ref) and torch.equal(hi, hi_ref)          # min / max are bit-exact in every test here
        lo_orc, hi_orc = _oracle_range(x, group)                            # ... and against the CPU oracle
        assert np.array_equal(_bits(lo), lo_orc.view(np.uint32)) and np.array_equal(_bits(hi), hi_orc.view(np.uint32))
        xf = x.float()
        if group == b.GROUP_CHANNEL:
            assert torch.equal(lo, xf.amin(dim=(0, 2, 3))) and torch.equal(hi, xf.amax(dim=(0, 2, 3)))


def test_too_many_groups_is_refused_before_anything_runs(b):
    n = b.NOALLOC_MAX_GROUPS + 1
    x = torch.zeros(1, n, 1, 4, device="cuda")
    lo = torch.full((n,), 7.0, device="cuda")
    hi = torch.full((n,), 7.0, device="cuda")
    with pytest.raises(b.GranqError) as err:
        b.granq_range_noalloc(x, lo, hi)
    assert err.value.status == b.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert bool((lo == 7.0).all()) and bool((hi == 7.0).all())               # outputs untouched
    # exactly at the limit it works
    x = torch.randn(1, b.NOALLOC_MAX_GROUPS, 1, 4, device="cuda")
    lo, hi, lo_ref, hi_ref = _pair(b, x, b.GROUP_CHANNEL)
    assert torch.equal(lo, lo_ref) and torch.equal(hi, hi_ref)
