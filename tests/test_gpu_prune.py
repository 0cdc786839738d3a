"""GPU pruning (nm_prune through the C ABI) against the CPU oracle: bit-exact indices and values."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_17301_b200 import inputs
from parity import assert_prune_bit_exact

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


def _check(nm, w, n, m, t):
    hnd = nm.nm_prune(w.cuda(), n, m, t)
    v, i = nm.nm_weights_export(hnd)
    torch.cuda.synchronize()
    vr, ir = oracle.prune(w.numpy(), n, m, t)
    assert_prune_bit_exact(v.cpu().numpy(), i.cpu().numpy(), vr, ir)
    assert (hnd.kk, hnd.n_tiles) == (vr.shape[1], ir.shape[0])
    return hnd


def test_tiny_config(nm):
    s = inputs.config_tiny()
    _check(nm, inputs.make_weights(s), s.n_keep, s.m_group, s.tile_t)


@pytest.mark.parametrize("s", inputs.config_resnet3x3(), ids=lambda s: s.name)
def test_resnet3x3_configs(nm, s):
    _check(nm, inputs.make_weights(s), s.n_keep, s.m_group, s.tile_t)


@pytest.mark.parametrize("s", inputs.config_bottleneck1x1(), ids=lambda s: s.name)
def test_bottleneck_configs(nm, s):
    _check(nm, inputs.make_weights(s), s.n_keep, s.m_group, s.tile_t)


@pytest.mark.parametrize("n,m,t,c_out,shape", [
    (3, 4, 5, 17, (5, 2, 5)),     # K = 50: tail group; tail tile
    (1, 8, 1, 9, (1, 1, 72)),     # T = 1: row-wise N:M
    (7, 16, 3, 10, (2, 5, 10)),
    (4, 4, 8, 24, (3, 3, 7)),     # N = M keeps everything
    (64, 128, 32, 64, (3, 3, 128)),   # adaptive-style large group
    (2, 4, 256, 512, (1, 1, 64)),
])
def test_odd_shapes(nm, n, m, t, c_out, shape):
    g = torch.Generator().manual_seed(n * 100 + m)
    w = torch.randn((c_out,) + shape, generator=g)
    _check(nm, w, n, m, t)


def test_ties_resolve_like_the_oracle(nm):
    g = torch.Generator().manual_seed(3)
    w = torch.randint(-2, 3, (32, 3, 3, 16), generator=g).float()  # few distinct scores: many ties
    _check(nm, w, 2, 4, 8)
    _check(nm, w, 1, 8, 4)
    _check(nm, torch.zeros(16, 1, 1, 32), 2, 4, 8)


def test_non_finite_weights_keep_n_per_group_and_match_the_oracle(nm):
    # a NaN score ranks as +infinity on both sides; no group keeps more than N, so nothing is
    # placed outside the index array (the placement is bounded as well)
    g = torch.Generator().manual_seed(9)
    w = torch.randn((40, 3, 3, 8), generator=g)
    flat = w.view(-1)
    pick = torch.randperm(flat.numel(), generator=g)[:60]
    flat[pick[:30]] = float("nan")
    flat[pick[30:45]] = float("inf")
    flat[pick[45:]] = float("-inf")
    w[39, 2, 2, 4:] = float("nan")                      # the last group of the last tile, whole
    for n, m, t in ((2, 4, 8), (1, 4, 16), (3, 8, 1), (2, 4, 64)):
        hnd = nm.nm_prune(w.cuda(), n, m, t)
        v, i = nm.nm_weights_export(hnd)
        torch.cuda.synchronize()
        vr, ir = oracle.prune(w.numpy(), n, m, t)
        assert np.array_equal(i.cpu().numpy(), ir)
        assert np.array_equal(v.cpu().numpy().view(np.uint32), vr.view(np.uint32))
        assert (ir.astype(np.int64) // m == np.arange(ir.shape[1]) // n).all()


def test_import_refuses_rows_without_the_group_structure(nm):
    # strictly ascending and below K, but three columns of the first group and one of the second
    s = inputs.config_tiny()
    hnd = nm.nm_prune(inputs.make_weights(s).cuda(), 2, 4, 8)
    v, i = nm.nm_weights_export(hnd)
    bad = i.cpu().view(torch.int16).clone()
    bad[1, 0:4] = torch.tensor([0, 1, 2, 5], dtype=torch.int16)
    with pytest.raises(nm.NmError) as e:
        nm.nm_weights_import(v, bad.view(torch.uint16).cuda(), 3, 3, 16, 2, 4, 8)
    assert e.value.status == nm.NM_ERR_INVALID_ARG
    assert "group" in str(e.value)


def test_import_round_trip_and_validation(nm):
    s = inputs.config_tiny()
    w = inputs.make_weights(s)
    hnd = _check(nm, w, 2, 4, 8)
    v, i = nm.nm_weights_export(hnd)
    h2 = nm.nm_weights_import(v, i, 3, 3, 16, 2, 4, 8)
    v2, i2 = nm.nm_weights_export(h2)
    assert torch.equal(v, v2) and torch.equal(i.view(torch.int16), i2.view(torch.int16))
    x = inputs.make_activations(s).cuda()
    y1 = nm.nm_conv2d(hnd, x, 3, 3, 1, 1, 1)
    y2 = nm.nm_conv2d(h2, x, 3, 3, 1, 1, 1)
    assert torch.equal(y1, y2)
    bad = i.clone().view(torch.int16)
    bad[0, 1] = bad[0, 0]
    with pytest.raises(nm.NmError) as e:
        nm.nm_weights_import(v, bad.view(torch.uint16), 3, 3, 16, 2, 4, 8)
    assert e.value.status == nm.NM_ERR_INVALID_ARG



def test_retained_l1_mass(nm):
    """Retained / total L1 mass against the plain sums over the oracle's result; wider tiles retain less."""
    import numpy as np
    import oracle
    g = torch.Generator().manual_seed(5)
    w = torch.randn((96, 3, 3, 32), generator=g)
    shares = []
    for t in (1, 8, 32, 96):
        hnd = nm.nm_prune(w.cuda(), 2, 4, t)
        kept, total = nm.nm_weights_retained_l1(hnd)
        vr, _ = oracle.prune(w.numpy(), 2, 4, t)
        assert total == pytest.approx(float(np.abs(w.numpy().astype(np.float64)).sum()), rel=1e-9)
        assert kept == pytest.approx(float(np.abs(vr.astype(np.float64)).sum()), rel=1e-9)
        shares.append(kept / total)
    assert shares == sorted(shares, reverse=True) and shares[0] > shares[-1]
    v, i = nm.nm_weights_export(nm.nm_prune(w.cuda(), 2, 4, 32))
    imported = nm.nm_weights_import(v, i, 3, 3, 32, 2, 4, 32)
    with pytest.raises(nm.NmError) as e:
        nm.nm_weights_retained_l1(imported)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
