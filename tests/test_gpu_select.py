"""The select kernel (plan.variant = 8: contraction over the retained columns only, kept columns picked in
registers under precomputed masks) against the CPU oracle, element by element: both forms of its activation
loads, every N:M pattern it covers, one to four tiles per work item, one to four MMA issuer threads, short
rings, several work items per CTA, blocks that span several images, split reduction axis."""
import numpy as np
import pytest
import torch

from paper_2507_17301_b200.inputs import ConvShape
from parity import assert_conv_close, assert_prune_bit_exact, gpu_layer, oracle_layer, tensors_for

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


def _plan(nm, **kw):
    p = nm.nm_plan_t()
    p.variant = 8
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def _plans(nm, s):
    t = s.tile_t
    return [_plan(nm), _plan(nm, loads=1), _plan(nm, loads=2), _plan(nm, bn=t), _plan(nm, bn=t, loads=1, stages=2),
            _plan(nm, bn=2 * t, issuers=1), _plan(nm, bn=4 * t, issuers=2, loads=1), _plan(nm, bn=4 * t, loads=2, stages=1), _plan(nm, loads=1, stages=4),
            _plan(nm, bn=256), _plan(nm, bn=128, loads=2),
            # four and eight epilogue warps (split = 1, 2; the default picks by the item's chunk count)
            _plan(nm, split=1), _plan(nm, split=2), _plan(nm, bn=t, split=2, loads=1), _plan(nm, bn=256, split=2), _plan(nm, bn=2 * t, split=1, issuers=2)]


# name, batch, h, w, c_in, c_out, kh, kw, stride, pad, dil, N, M, T
SHAPES = [
    ConvShape("sel_3x3", 2, 16, 16, 64, 64, 3, 3, 1, 1, 1, 2, 4, 32),
    ConvShape("sel_ragged", 3, 13, 13, 128, 64, 3, 3, 1, 1, 1, 2, 4, 32),            # 507 pixels: ragged last block
    ConvShape("sel_stride2", 2, 15, 15, 128, 64, 3, 3, 2, 1, 1, 2, 4, 32),          # im2col loads only
    ConvShape("sel_nopad", 2, 20, 20, 64, 32, 3, 3, 1, 0, 1, 2, 4, 16),             # output smaller than input: im2col only
    ConvShape("sel_dil2", 2, 20, 20, 64, 32, 3, 3, 1, 2, 2, 2, 4, 16),              # dilated, same size: patch form with a wide halo
    ConvShape("sel_1x1", 2, 14, 14, 256, 96, 1, 1, 1, 0, 1, 2, 4, 32),
    ConvShape("sel_1x1_s2", 2, 14, 14, 256, 64, 1, 1, 2, 0, 1, 1, 4, 64),
    ConvShape("sel_5x5", 1, 24, 24, 64, 32, 5, 5, 1, 2, 1, 2, 8, 16),               # 25 taps
    ConvShape("sel_7x7_images", 5, 7, 7, 256, 64, 3, 3, 1, 1, 1, 2, 4, 64),         # a block spans three images
    ConvShape("sel_1of4", 2, 15, 15, 128, 128, 3, 3, 1, 1, 1, 1, 4, 64),
    ConvShape("sel_3of4", 2, 16, 16, 96, 64, 3, 3, 1, 1, 1, 3, 4, 64),              # chunks of 32 source columns
    ConvShape("sel_1of8", 1, 16, 16, 128, 64, 3, 3, 1, 1, 1, 1, 8, 64),
    ConvShape("sel_2of8", 2, 15, 15, 128, 128, 3, 3, 1, 1, 1, 2, 8, 32),
    ConvShape("sel_4of8", 1, 20, 20, 128, 64, 1, 1, 1, 0, 1, 4, 8, 16),
    ConvShape("sel_tile128", 1, 16, 16, 128, 256, 3, 3, 1, 1, 1, 2, 4, 128),
    ConvShape("sel_tile256", 1, 16, 16, 128, 512, 1, 1, 1, 0, 1, 2, 4, 256),
    ConvShape("sel_tile256_3x3", 3, 14, 14, 64, 256, 3, 3, 1, 1, 1, 2, 4, 256),
    ConvShape("sel_many_items", 8, 56, 56, 64, 64, 3, 3, 1, 1, 1, 2, 4, 64),        # 196 work items: two per CTA, widest halo
    ConvShape("sel_wide", 2, 28, 28, 64, 512, 1, 1, 1, 0, 1, 2, 4, 64),             # 4 tiles per item, 2 channel slices
    ConvShape("sel_asym", 2, 18, 22, 64, 32, 3, 5, 1, 1, 1, 2, 4, 16),              # 3x5 kernel: im2col only (pad 1 does not keep the width)
]


def _run(nm, s, integer):
    w, x, b = tensors_for(s, integer)
    vr, ir, yr = oracle_layer(s, w, x, b)
    ran, patch_ran = 0, 0
    for plan in _plans(nm, s):
        try:
            _, v, i, y = gpu_layer(nm, s, w, x, b, True, plan)
        except nm.NmError as e:
            if e.status == nm.NM_ERR_UNSUPPORTED:
                continue
            raise
        ran += 1
        patch_ran += plan.loads == 2
        assert_prune_bit_exact(v, i, vr, ir)
        if integer:
            assert np.array_equal(y, yr), f"integer case differs: {plan.as_dict()}"
        else:
            assert_conv_close(y, yr)
    assert ran >= 3, f"the select kernel took {s.name} with {ran} plans only"
    same_size = s.stride == 1 and 2 * s.pad == s.dil * (s.kh - 1) and 2 * s.pad == s.dil * (s.kw - 1)
    assert (patch_ran > 0) == same_size


@pytest.mark.parametrize("s", SHAPES, ids=lambda s: s.name)
def test_select_kernel_integer_exact(nm, s):
    _run(nm, s, True)


@pytest.mark.parametrize("s", SHAPES, ids=lambda s: s.name)
def test_select_kernel(nm, s):
    _run(nm, s, False)


@pytest.mark.parametrize("integer", [False, True], ids=["normal", "integer_exact"])
@pytest.mark.parametrize("loads", [1, 2])
def test_select_kernel_split_reduction_axis(nm, integer, loads):
    """Few pixel blocks and a long reduction axis: ranges of the axis go to different CTAs, the partial sums
    through the handle's scratch and a second pass."""
    s = ConvShape("sel_splitk", 2, 14, 14, 256, 64, 3, 3, 1, 1, 1, 2, 4, 32)       # 4 channel blocks of 64 x 9 taps
    w, x, b = tensors_for(s, integer)
    vr, ir, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd = x.cuda(), b.cuda()
    plan = _plan(nm, bn=64, ksplit=2, loads=loads)
    with pytest.raises(nm.NmError) as e:                      # no scratch yet: the plan is refused
        nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    need = nm.nm_plan_scratch_bytes(hnd, xd.shape, s.stride, s.pad, s.dil, _plan(nm, bn=64, ksplit=4))
    assert need == 4 * 512 * 64 * 4
    nm.nm_weights_reserve(hnd, need)
    for ksplit in (2, 4) + ((3,) if loads == 1 else ()):      # patch form: 4 channel blocks; im2col: 36 chunks
        for bn in (32, 64):
            plan = _plan(nm, bn=bn, ksplit=ksplit, loads=loads)
            for _ in range(2):                                # twice: the scratch is reused
                y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
            nm.nm_weights_check(hnd)
            torch.cuda.synchronize()
            if integer:
                assert np.array_equal(y.cpu().numpy(), yr), (ksplit, bn)
            else:
                assert_conv_close(y.cpu().numpy(), yr)


def test_select_kernel_with_shortcut(nm):
    """act(conv + bias + residual) through the select kernel's epilogue and through its split form."""
    import oracle
    s = ConvShape("sel_res", 3, 14, 14, 128, 128, 3, 3, 1, 1, 1, 2, 4, 64)
    g = torch.Generator().manual_seed(5)
    w = torch.randint(-3, 4, (s.c_out, 3, 3, s.c_in), generator=g).float()
    x = torch.randint(-3, 4, (s.batch, s.h, s.w, s.c_in), generator=g).float()
    b = torch.randint(-3, 4, (s.c_out,), generator=g).float()
    res = torch.randint(-9, 10, (s.batch, s.h, s.w, s.c_out), generator=g).float()
    vr, ir = oracle.prune(w.numpy(), 2, 4, 64)
    yr = oracle.conv2d_res(vr, ir, 3, 3, s.c_in, 64, x.numpy(), (1, 1), (1, 1), (1, 1), b.numpy(), res.numpy(), True)
    hnd = nm.nm_prune(w.cuda(), 2, 4, 64)
    nm.nm_weights_reserve(hnd, 2 * 640 * 128 * 4)
    for plan in (_plan(nm), _plan(nm, loads=1, bn=64), _plan(nm, ksplit=2), _plan(nm, split=1), _plan(nm, split=2)):
        y = nm.nm_conv2d(hnd, x.cuda(), 3, 3, 1, 1, 1, b.cuda(), True, plan=plan, residual=res.cuda())
        nm.nm_weights_check(hnd)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), yr), plan.as_dict()
