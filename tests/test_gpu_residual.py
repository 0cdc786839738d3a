"""nm_conv2d_res (shortcut addition fused into the epilogue) against the oracle's shortcut-adding form,
through every kernel variant that takes the shape."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_17301_b200.inputs import ConvShape
from parity import assert_conv_close, tensors_for
from test_gpu_conv import _plans

pytestmark = pytest.mark.gpu

SHAPES = [
    ConvShape("res_small_3x3", 2, 9, 11, 16, 24, 3, 3, 1, 1, 1, 2, 4, 8),                 # gather / slab kernels
    ConvShape("res_1x1_ragged", 3, 13, 13, 96, 64, 1, 1, 1, 0, 1, 2, 4, 32),              # 507 pixels: ragged last block
    ConvShape("res_3x3_window", 2, 28, 28, 64, 64, 3, 3, 1, 1, 1, 2, 4, 32),
    ConvShape("res_stride2", 2, 15, 15, 128, 64, 3, 3, 2, 1, 1, 2, 4, 32),
    ConvShape("res_few_channels", 2, 32, 32, 3, 64, 7, 7, 2, 3, 1, 1, 1, 64),             # row-run kernel
    ConvShape("res_long_k", 2, 14, 14, 256, 64, 3, 3, 1, 1, 1, 2, 4, 32),                 # split-K and balanced plans after tuning
    ConvShape("res_pw_cout24", 2, 56, 56, 96, 24, 1, 1, 1, 0, 1, 2, 4, 8),                # pointwise, channels end inside a 32-block
    ConvShape("res_pw_cin24_cout144", 1, 56, 56, 24, 144, 1, 1, 1, 0, 1, 2, 4, 16),
]


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


@pytest.mark.parametrize("integer", [False, True], ids=["normal", "integer_exact"])
@pytest.mark.parametrize("s", SHAPES, ids=lambda s: s.name)
def test_residual_epilogue(nm, s, integer):
    w, x, b = tensors_for(s, integer)
    g = torch.Generator().manual_seed(91)
    shape = (s.batch, s.ho, s.wo, s.c_out)
    res = torch.randint(-6, 7, shape, generator=g).float() if integer else torch.randn(shape, generator=g)
    vr, ir = oracle.prune(w.numpy(), s.n_keep, s.m_group, s.tile_t)
    yr = oracle.conv2d_res(vr, ir, s.kh, s.kw, s.c_in, s.tile_t, x.numpy(), (s.stride,) * 2, (s.pad,) * 2, (s.dil,) * 2,
                           b.numpy(), res.numpy(), True)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd, rd = x.cuda(), b.cuda(), res.cuda()
    nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, True, kh=s.kh, kw=s.kw)    # reserves split-K scratch if any
    plans = _plans(nm, s)
    for splits, kblk, issuers in ((2, 0, 0), (3, 0, 0), (-1, 0, 0), (-1, 2, 0), (2, 0, 2), (-1, 0, 2)):   # split-K, and balanced ranges (need the tuner's scratch)
        p = nm.nm_plan_t()
        p.variant, p.bn, p.split, p.kblk, p.issuers = 4, 64, splits, kblk, issuers
        plans.append(p)
    ran = set()
    for plan in plans:
        try:
            y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, True, plan=plan, residual=rd)
        except nm.NmError as e:
            if plan is not None and e.status == nm.NM_ERR_UNSUPPORTED:
                continue
            raise
        nm.nm_weights_check(hnd)
        torch.cuda.synchronize()
        ran.add((plan.variant, plan.split) if plan is not None else (0, 0))
        if integer:
            assert np.array_equal(y.cpu().numpy(), yr), f"plan {plan.as_dict() if plan else None}"
        else:
            assert_conv_close(y.cpu().numpy(), yr)
    assert len(ran) >= 2
    # without a residual the entry point is nm_conv2d
    y0 = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, True)
    y1 = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, True, residual=torch.zeros_like(rd))
    torch.cuda.synchronize()
    assert torch.equal(y0, y1)


def test_residual_argument_errors(nm):
    s = SHAPES[0]
    w, x, b = tensors_for(s)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    bad = torch.zeros(s.batch * s.ho * s.wo * s.c_out + 1, device="cuda")[1:].view(s.batch, s.ho, s.wo, s.c_out)
    with pytest.raises(nm.NmError) as e:
        nm.nm_conv2d(hnd, x.cuda(), s.kh, s.kw, s.stride, s.pad, s.dil, b.cuda(), True, residual=bad)
    assert e.value.status == nm.NM_ERR_INVALID_ARG


def test_chained_block_matches_oracle_chain(nm):
    """A small residual block chained on the device (conv -> max-pool -> 1x1 -> 3x3 -> 1x1 + shortcut) against the
    same chain of oracle calls: each layer consumes the previous layer's device output."""
    g = torch.Generator().manual_seed(17)
    x = torch.randn((2, 32, 32, 3), generator=g)
    ws = [torch.randn(sh, generator=g) * sc for sh, sc in (((64, 7, 7, 3), 0.08), ((32, 1, 1, 64), 0.15),
                                                            ((32, 3, 3, 32), 0.08), ((64, 1, 1, 32), 0.2))]
    nms = [(1, 1, 64), (2, 4, 32), (2, 4, 32), (2, 4, 32)]
    hs = [nm.nm_prune(w.cuda(), n, m, t) for w, (n, m, t) in zip(ws, nms)]
    pr = [oracle.prune(w.numpy(), n, m, t) for w, (n, m, t) in zip(ws, nms)]
    # device chain
    a = nm.nm_conv2d(hs[0], x.cuda(), 7, 7, 2, 3, 1, None, True)
    p0 = nm.nm_maxpool2d(a, 3, 2, 1)
    t = nm.nm_conv2d(hs[1], p0, 1, 1, 1, 0, 1, None, True)
    t = nm.nm_conv2d(hs[2], t, 3, 3, 1, 1, 1, None, True)
    out = nm.nm_conv2d(hs[3], t, 1, 1, 1, 0, 1, None, True, residual=p0)
    torch.cuda.synchronize()
    # oracle chain
    ra = oracle.conv2d(pr[0][0], pr[0][1], 7, 7, 3, 64, x.numpy(), (2, 2), (3, 3), (1, 1), None, True)
    rp = oracle.maxpool2d(ra, (3, 3), (2, 2), (1, 1))
    rt = oracle.conv2d(pr[1][0], pr[1][1], 1, 1, 64, 32, rp, (1, 1), (0, 0), (1, 1), None, True)
    rt = oracle.conv2d(pr[2][0], pr[2][1], 3, 3, 32, 32, rt, (1, 1), (1, 1), (1, 1), None, True)
    ro = oracle.conv2d_res(pr[3][0], pr[3][1], 1, 1, 32, 32, rt, (1, 1), (0, 0), (1, 1), None, rp, True)
    assert_conv_close(out.cpu().numpy(), ro)
