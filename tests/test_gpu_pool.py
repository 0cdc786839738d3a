"""nm_maxpool2d against the oracle (bit-exact: a maximum has no rounding)."""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


@pytest.mark.parametrize("shape,kernel,stride,pad", [
    ((2, 112, 112, 64), 3, 2, 1),          # the ResNet stem's pooling at its real size (two images)
    ((3, 17, 13, 8), 3, 2, 1),             # ragged sizes
    ((1, 9, 9, 4), (2, 3), (1, 2), (0, 1)),
    ((2, 8, 8, 12), 2, 2, 0),
])
def test_maxpool_matches_oracle(nm, shape, kernel, stride, pad):
    g = torch.Generator().manual_seed(2)
    x = torch.randn(shape, generator=g)
    pair = lambda v: (v, v) if isinstance(v, int) else v
    want = oracle.maxpool2d(x.numpy(), pair(kernel), pair(stride), pair(pad))
    got = nm.nm_maxpool2d(x.cuda(), kernel, stride, pad)
    torch.cuda.synchronize()
    assert np.array_equal(got.cpu().numpy(), want)


def test_maxpool_argument_errors(nm):
    x = torch.zeros((1, 8, 8, 6), device="cuda")
    with pytest.raises(nm.NmError) as e:
        nm.nm_maxpool2d(x, 3, 2, 1)                    # channels not a multiple of 4
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    with pytest.raises(nm.NmError) as e:
        nm.nm_maxpool2d(torch.zeros((1, 8, 8, 8), device="cuda"), 2, 2, 2)   # padding as large as the window
    assert e.value.status == nm.NM_ERR_INVALID_ARG
