"""Layers of the benchmark workload at the benchmark's own size (ResNet-50 shapes, batch 64) and in its
launch configuration (the plan nm_autotune picks), checked on sampled outputs: whole images of the
batch that the CPU oracle computes one by one."""
import numpy as np
import pytest
import torch

import oracle
from paper_2507_17301_b200 import inputs
from parity import assert_conv_close, assert_prune_bit_exact

pytestmark = pytest.mark.gpu

# stem (dense, few channels), 1x1 wide output, 3x3 at 56x56, strided 3x3, strided 1x1 projection,
# tensor-bound 3x3 at 14x14, long-reduction 1x1 and 3x3 at 7x7 (split-K candidates)
LAYERS = [(50, "stem7x7"), (50, "s1b1_c3"), (50, "s1b1_c2"), (50, "s2b1_c2"), (50, "s2b1_ds"), (50, "s3b2_c2"),
          (50, "s4b2_c1"), (50, "s4b2_c2"),
          # basic-block network (ResNet-34): strided 3x3 that doubles the channels, 3x3 at 28x28
          (34, "s2b1_c1"), (34, "s2b2_c2")]
# pointwise layers of MobileNet-V2 (tile width 16): channel counts that are not multiples of 32 on either
# side (general kernels), the widest expansion, the last 1x1
MOBILE_LAYERS = ["b1r1_project", "b2r2_expand", "b3r1_project", "b5r2_expand", "b6r2_project", "last_1x1"]
IMAGES = (0, 37, 63)


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


@pytest.fixture(scope="module")
def stack():
    return {depth: {s.name: (i, s) for i, s in enumerate(inputs.resnet_conv_stack(depth, 64, 2, 4, tile_t=64))}
            for depth in (34, 50)}


@pytest.mark.parametrize("depth,name", LAYERS, ids=[f"r{d}_{n}" for d, n in LAYERS])
def test_stack_layer_sampled_images(nm, stack, depth, name):
    li, s = stack[depth][name]
    w = inputs.make_weights(s, li)
    b = inputs.make_bias(s, li)
    g = torch.Generator().manual_seed(1 + 1000 * li)
    x = torch.randn((s.batch, s.h, s.w, s.c_in), generator=g)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    v, i = nm.nm_weights_export(hnd)
    vr, ir = oracle.prune(w.numpy(), s.n_keep, s.m_group, s.tile_t)
    assert_prune_bit_exact(v.cpu().numpy(), i.cpu().numpy(), vr, ir)
    xd, bd = x.cuda(), b.cuda()
    plan, ms = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)
    assert ms > 0
    y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
    nm.nm_weights_check(hnd)
    torch.cuda.synchronize()
    for n in IMAGES:
        yr = oracle.conv2d(vr, ir, s.kh, s.kw, s.c_in, s.tile_t, x[n:n + 1].numpy(), (s.stride,) * 2, (s.pad,) * 2,
                           (s.dil,) * 2, b.numpy(), s.relu)
        assert_conv_close(y[n:n + 1].cpu().numpy(), yr)
    # the rest of the batch: finite everywhere, and no image left unwritten (a ReLU layer may hold zeros,
    # an all-zero image would mean a skipped work item)
    yc = y.cpu()
    assert torch.isfinite(yc).all()
    assert (yc.abs().amax(dim=(1, 2, 3)) > 0).all()


# Configuration 5 of the workload list: ResNet-101 shapes at batch 128 under 1:4 and under 2:8, plans from
# nm_autotune, sampled whole images.  One layer of each kind: 3x3 at 14x14 (tensor-bound), 1x1 at 56x56 (wide
# output), the stem, a strided projection, and a long-reduction layer at 7x7 (few work items: split or balanced plans).
R101_LAYERS = ["stem7x7", "s1b1_c3", "s3b2_c2", "s3b1_ds", "s4b2_c1"]
R101_IMAGES = (0, 64, 127)


@pytest.fixture(scope="module")
def stack101():
    return {(n, m): {s.name: (i, s) for i, s in enumerate(inputs.resnet_conv_stack(101, 128, n, m, tile_t=64))}
            for n, m in ((1, 4), (2, 8))}


def _sampled_layer(nm, li, s, images):
    w = inputs.make_weights(s, li)
    b = inputs.make_bias(s, li)
    g = torch.Generator().manual_seed(1 + 1000 * li)
    x = torch.empty((s.batch, s.h, s.w, s.c_in))
    for b0 in range(0, s.batch, 16):   # drawn in slices: the stem's batch-128 input is 77 M floats
        x[b0:b0 + 16] = torch.randn((min(16, s.batch - b0), s.h, s.w, s.c_in), generator=g)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    v, i = nm.nm_weights_export(hnd)
    vr, ir = oracle.prune(w.numpy(), s.n_keep, s.m_group, s.tile_t)
    assert_prune_bit_exact(v.cpu().numpy(), i.cpu().numpy(), vr, ir)
    xd, bd = x.cuda(), b.cuda()
    plan, ms = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)
    assert ms > 0
    y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
    nm.nm_weights_check(hnd)
    torch.cuda.synchronize()
    for n in images:
        yr = oracle.conv2d(vr, ir, s.kh, s.kw, s.c_in, s.tile_t, x[n:n + 1].numpy(), (s.stride,) * 2, (s.pad,) * 2,
                           (s.dil,) * 2, b.numpy(), s.relu)
        assert_conv_close(y[n:n + 1].cpu().numpy(), yr)
    assert torch.isfinite(y).all()
    assert (y.abs().amax(dim=(1, 2, 3)) > 0).all()
    return plan


@pytest.mark.parametrize("name", R101_LAYERS)
@pytest.mark.parametrize("pattern", [(1, 4), (2, 8)], ids=["1of4", "2of8"])
def test_resnet101_batch128_sampled_images(nm, stack101, pattern, name):
    li, s = stack101[pattern][name]
    _sampled_layer(nm, li, s, R101_IMAGES)


# Configuration 3: the three bottleneck 1x1 shapes at their full batch of 64 under 2:4 and 1:8.
@pytest.mark.parametrize("s", inputs.config_bottleneck1x1(), ids=lambda s: s.name)
def test_bottleneck1x1_batch64_sampled_images(nm, s):
    assert s.batch == 64
    _sampled_layer(nm, 0, s, IMAGES)


@pytest.fixture(scope="module")
def mobile_stack():
    return {s.name: (i, s) for i, s in enumerate(inputs.mobilenet_v2_pointwise(64, 2, 4, tile_t=16))}


@pytest.mark.parametrize("name", MOBILE_LAYERS)
def test_mobilenet_pointwise_sampled_images(nm, mobile_stack, name):
    li, s = mobile_stack[name]
    w = inputs.make_weights(s, li)
    b = inputs.make_bias(s, li)
    g = torch.Generator().manual_seed(1 + 1000 * li)
    x = torch.randn((s.batch, s.h, s.w, s.c_in), generator=g)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    v, i = nm.nm_weights_export(hnd)
    vr, ir = oracle.prune(w.numpy(), s.n_keep, s.m_group, s.tile_t)
    assert_prune_bit_exact(v.cpu().numpy(), i.cpu().numpy(), vr, ir)
    xd, bd = x.cuda(), b.cuda()
    plan, ms = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)
    assert ms > 0
    for use in (plan, None):                                  # the tuned plan and the library default
        y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=use)
        nm.nm_weights_check(hnd)
        torch.cuda.synchronize()
        for n in IMAGES[:2]:
            yr = oracle.conv2d(vr, ir, s.kh, s.kw, s.c_in, s.tile_t, x[n:n + 1].numpy(), (s.stride,) * 2, (s.pad,) * 2,
                               (s.dil,) * 2, b.numpy(), s.relu)
            assert_conv_close(y[n:n + 1].cpu().numpy(), yr)
        assert torch.isfinite(y).all()

