"""GPU convolution (nm_conv2d through the C ABI) against the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2507_17301_b200 import inputs
from paper_2507_17301_b200.inputs import ConvShape
from parity import (assert_conv_close, assert_prune_bit_exact, errors, gpu_layer, oracle_layer, tensors_for)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


def _plans(nm, s):
    """Every kernel variant that admits the shape, plus the library default."""
    out = [None]
    for variant, split in ((1, 0), (2, 0), (2, 1)):   # split = 1: slab kernel with its cp.async producer
        p = nm.nm_plan_t()
        p.variant, p.split = variant, split
        out.append(p)
    # stream kernel: default width, 256 channels per CTA (one accumulator buffer), one tile per CTA,
    # and a two-stage ring (every stage reused many times)
    for bn, stages in ((0, 0), (256, 0), (s.tile_t if s is not None else 16, 0), (0, 2)):
        p = nm.nm_plan_t()
        p.variant, p.bn, p.stages = 3, bn, stages
        out.append(p)
    # expanded-operand kernel: default width, 32 and 256 channels per work item, two-stage ring, and
    # (split = 1) weights streamed per stage instead of kept resident
    for bn, stages, split, kblk in ((0, 0, 0, 0), (32, 0, 0, 0), (256, 0, 0, 0), (0, 2, 0, 0), (0, 0, 1, 0), (64, 0, 1, 0),
                                    (0, 0, 0, 2), (128, 2, 1, 2), (256, 0, 1, 2)):   # kblk = 2: two 32-column blocks per stage
        p = nm.nm_plan_t()
        p.variant, p.bn, p.stages, p.split, p.kblk = 4, bn, stages, split, kblk
        out.append(p)
    # one and two MMA issuer threads (two: alternate stages, an accumulator each; one accumulator buffer at 256 channels),
    # with weights resident / streamed, one and two blocks per stage, a two-stage ring
    for bn, issuers, split, kblk, stages in ((0, 1, 0, 0, 0), (128, 1, 0, 0, 0), (64, 2, 0, 0, 0), (256, 2, 0, 0, 0), (32, 2, 0, 0, 0),
                                             (0, 2, 1, 2, 0), (256, 2, 1, 1, 2), (128, 2, 1, 2, 2), (64, 2, 1, 1, 4)):
        p = nm.nm_plan_t()
        p.variant, p.bn, p.issuers, p.split, p.kblk, p.stages = 4, bn, issuers, split, kblk, stages
        out.append(p)
    p = nm.nm_plan_t()
    p.variant = 5                                     # row-run kernel
    out.append(p)
    # plane kernel: as many output rows per item as fit, two rows with two band buffers, one row, three rows
    for rows, stages in ((0, 0), (2, 2), (1, 0), (3, 3)):
        p = nm.nm_plan_t()
        p.variant, p.split, p.stages = 9, rows, stages
        out.append(p)
    # window kernel: default, one M-tile with 64 channels, two / three / four M-tiles, short weight ring
    for bn, mt, stages in ((0, 0, 0), (64, 1, 0), (0, 2, 0), (32, 1, 3), (64, 3, 0), (32, 4, 0), (128, 4, 0)):
        p = nm.nm_plan_t()
        p.variant, p.bn, p.split, p.stages = 6, bn, mt, stages
        out.append(p)
    # pair kernel (clusters of two CTAs): default, both widths, a two-stage ring
    for bn, stages, kblk in ((0, 0, 0), (128, 0, 1), (256, 0, 1), (128, 2, 2)):
        p = nm.nm_plan_t()
        p.variant, p.bn, p.stages, p.kblk = 7, bn, stages, kblk
        out.append(p)
    return out


def _run(nm, s, integer=False, use_bias=True, need_variant=None):
    w, x, b = tensors_for(s, integer)
    vr, ir, yr = oracle_layer(s, w, x, b, use_bias)
    ran = 0
    variants_run = set()
    for plan in _plans(nm, s):
        try:
            _, v, i, y = gpu_layer(nm, s, w, x, b, use_bias, plan)
        except nm.NmError as e:
            if plan is not None and e.status == nm.NM_ERR_UNSUPPORTED:
                continue  # this variant does not take the shape
            raise
        ran += 1
        variants_run.add(plan.variant if plan is not None else 0)
        assert_prune_bit_exact(v, i, vr, ir)
        if integer:
            # every product and partial sum is exact in TF32 / fp32: results must be identical
            assert np.array_equal(y, yr), f"integer case differs (variant {plan.variant if plan else 0})"
        else:
            assert_conv_close(y, yr)
    assert ran >= 2  # the default and at least one explicit variant
    for v in need_variant or ():
        assert v in variants_run, f"variant {v} did not take {s.name}"


def test_tiny_config(nm):
    _run(nm, inputs.config_tiny())


def test_tiny_config_integer_exact(nm):
    _run(nm, inputs.config_tiny(), integer=True)


SMALL = [
    ConvShape("s1_3x3_T8", 2, 9, 11, 16, 24, 3, 3, 1, 1, 1, 2, 4, 8),
    ConvShape("ragged_pixels", 3, 13, 13, 32, 32, 3, 3, 1, 1, 1, 2, 4, 32),        # 507 pixels: 3 full tiles + tail
    ConvShape("stride2", 2, 15, 15, 32, 64, 3, 3, 2, 1, 1, 2, 4, 32),
    ConvShape("dilation2", 1, 12, 12, 16, 16, 3, 3, 1, 2, 2, 1, 4, 16),
    ConvShape("one_by_one", 2, 7, 7, 64, 48, 1, 1, 1, 0, 1, 2, 4, 16),
    ConvShape("one_by_one_s2", 2, 14, 14, 64, 32, 1, 1, 2, 0, 1, 1, 8, 32),
    ConvShape("tail_tile", 1, 8, 8, 16, 40, 3, 3, 1, 1, 1, 2, 4, 16),               # c_out % T != 0
    ConvShape("tail_group", 1, 8, 8, 6, 8, 3, 3, 1, 1, 1, 3, 4, 8),                 # K = 54, c_in % 4 != 0
    ConvShape("t1_rowwise", 1, 6, 6, 16, 12, 3, 3, 1, 1, 1, 2, 4, 1),               # T = 1
    ConvShape("odd_tile", 1, 6, 6, 16, 21, 1, 1, 1, 0, 1, 2, 4, 7),                 # T = 7
    ConvShape("keep_all", 1, 10, 10, 8, 16, 3, 3, 1, 1, 1, 4, 4, 16),               # N = M: dense
    ConvShape("stem_like", 1, 32, 32, 3, 64, 7, 7, 2, 3, 1, 1, 1, 64),              # 7x7, c_in = 3, dense
    ConvShape("big_tile", 1, 12, 12, 64, 256, 3, 3, 1, 1, 1, 2, 8, 128),
    ConvShape("tile256", 1, 12, 12, 32, 256, 1, 1, 1, 0, 1, 1, 4, 256),
    ConvShape("no_pad_5x5", 1, 11, 11, 8, 8, 5, 5, 1, 0, 1, 2, 4, 8),
    ConvShape("single_pixel", 1, 3, 3, 16, 16, 3, 3, 1, 0, 1, 2, 4, 16),            # one output pixel
]


@pytest.mark.parametrize("s", SMALL, ids=lambda s: s.name)
def test_small_shapes(nm, s):
    _run(nm, s)


# inputs of at least 128 KiB with c_in % 32 == 0: these take the TMA (im2col) producer
MEDIUM = [
    ConvShape("tma_3x3", 2, 16, 16, 64, 64, 3, 3, 1, 1, 1, 2, 4, 32),
    ConvShape("tma_ragged_tail", 3, 13, 13, 96, 64, 3, 3, 1, 1, 1, 2, 4, 64),      # 507 pixels
    ConvShape("tma_stride2", 2, 15, 15, 128, 64, 3, 3, 2, 1, 1, 2, 4, 32),
    ConvShape("tma_dilation2", 1, 20, 20, 96, 32, 3, 3, 1, 2, 2, 2, 4, 32),
    ConvShape("tma_1x1", 2, 14, 14, 256, 96, 1, 1, 1, 0, 1, 2, 4, 32),
    ConvShape("tma_1x1_stride2", 2, 14, 14, 256, 64, 1, 1, 2, 0, 1, 1, 4, 64),
    ConvShape("tma_5x5", 1, 24, 24, 64, 32, 5, 5, 1, 2, 1, 2, 8, 16),
    ConvShape("tma_tile8", 2, 16, 16, 64, 24, 3, 3, 1, 1, 1, 2, 4, 8),
    ConvShape("tma_1of8", 1, 16, 16, 128, 64, 3, 3, 1, 1, 1, 1, 8, 64),
    ConvShape("tma_3of4", 1, 16, 16, 128, 64, 1, 1, 1, 0, 1, 3, 4, 64),
    ConvShape("tma_dense", 1, 16, 16, 128, 48, 3, 3, 1, 1, 1, 4, 4, 16),
    ConvShape("tma_tile128", 1, 16, 16, 128, 256, 3, 3, 1, 1, 1, 2, 4, 128),
    ConvShape("tma_dense_64", 1, 16, 16, 128, 64, 3, 3, 1, 1, 1, 4, 4, 32),
    ConvShape("tma_tile256", 1, 16, 16, 128, 512, 1, 1, 1, 0, 1, 2, 4, 256),
    ConvShape("tma_1of4", 2, 15, 15, 96, 128, 3, 3, 1, 1, 1, 1, 4, 64),
    ConvShape("tma_2of8", 2, 15, 15, 128, 128, 3, 3, 1, 1, 1, 2, 8, 32),
    ConvShape("tma_4of8", 1, 20, 20, 128, 64, 1, 1, 1, 0, 1, 4, 8, 16),
    ConvShape("tma_cin32_3x3", 2, 20, 20, 32, 64, 3, 3, 1, 1, 1, 2, 4, 16),          # K = 288: half-filled last chunk
    ConvShape("tma_many_items", 8, 56, 56, 32, 128, 1, 1, 1, 0, 1, 2, 4, 64),        # 196 work items: several per CTA
    ConvShape("tma_many_items_3x3", 4, 56, 56, 32, 64, 3, 3, 1, 1, 1, 2, 4, 32),     # 196 work items of 5 chunks, last chunk half-filled
    ConvShape("tma_wide_256", 2, 28, 28, 64, 512, 1, 1, 1, 0, 1, 2, 4, 64),          # 4 tiles per CTA at bn = 256
]


# few input channels, c_out a multiple of 32, dil_w = 1, output rows of at most 128 pixels: row-run kernel
ROWRUN = [
    ConvShape("rr_stem", 2, 64, 64, 3, 64, 7, 7, 2, 3, 1, 1, 1, 64),
    ConvShape("rr_stem_wide", 1, 40, 252, 3, 32, 7, 7, 2, 3, 1, 1, 1, 32),          # 126 output pixels per row
    ConvShape("rr_3x3_c4", 2, 20, 20, 4, 64, 3, 3, 1, 1, 1, 2, 4, 8),                # pruned, tile 8
    ConvShape("rr_5x5_c8_s1", 1, 30, 30, 8, 64, 5, 5, 1, 2, 1, 2, 4, 32),
    ConvShape("rr_nopad", 1, 24, 24, 4, 32, 3, 3, 1, 0, 1, 4, 4, 32),
    ConvShape("rr_1x1_c12", 3, 10, 16, 12, 128, 1, 1, 1, 0, 1, 1, 4, 16),
    ConvShape("rr_k500", 2, 12, 12, 20, 32, 5, 5, 2, 2, 1, 2, 4, 32),                # K = 500: 16 sub-tiles
]


@pytest.mark.parametrize("s", ROWRUN, ids=lambda s: s.name)
def test_rowrun_shapes(nm, s):
    _run(nm, s, need_variant=[5])


@pytest.mark.parametrize("s", ROWRUN[:4], ids=lambda s: s.name)
def test_rowrun_shapes_integer_exact(nm, s):
    _run(nm, s, integer=True, need_variant=[5])


# at most four input channels, horizontal stride 1 or 2, kernel rows of at most 8 taps: plane kernel
PLANES = [
    ConvShape("pl_stem", 2, 64, 64, 3, 64, 7, 7, 2, 3, 1, 1, 1, 64),
    ConvShape("pl_stem_wide", 1, 40, 252, 3, 32, 7, 7, 2, 3, 1, 1, 1, 32),          # 126 output pixels per row
    ConvShape("pl_ragged_band", 3, 30, 50, 3, 64, 7, 7, 2, 3, 1, 1, 1, 64),         # 15 output rows: a last band of three
    ConvShape("pl_3x3_c4_s1", 2, 20, 20, 4, 64, 3, 3, 1, 1, 1, 2, 4, 8),             # stride 1, pruned, tile 8
    ConvShape("pl_nopad_s1", 1, 24, 24, 4, 32, 3, 3, 1, 0, 1, 4, 4, 32),
    ConvShape("pl_c1_5x5", 2, 31, 31, 1, 32, 5, 5, 2, 2, 1, 1, 1, 32),               # one channel, odd sizes
    ConvShape("pl_c2_3x8", 1, 18, 40, 2, 128, 3, 8, 2, 3, 1, 1, 1, 32),              # eight taps per kernel row, two rows per item
    ConvShape("pl_c256", 1, 16, 16, 3, 256, 3, 3, 1, 1, 1, 1, 1, 64),                # 256 channels: one output row per item
    ConvShape("pl_stem_224", 1, 224, 224, 3, 64, 7, 7, 2, 3, 1, 1, 1, 64),           # the ResNet stem at full size
]


@pytest.mark.parametrize("s", PLANES, ids=lambda s: s.name)
def test_plane_shapes(nm, s):
    _run(nm, s, need_variant=[9])


@pytest.mark.parametrize("s", PLANES[:8], ids=lambda s: s.name)
def test_plane_shapes_integer_exact(nm, s):
    _run(nm, s, integer=True, need_variant=[9])


# stride-1 spatial kernels with c_in and c_out multiples of 32: window kernel
WINDOW = [
    ConvShape("win_3x3_56", 1, 56, 56, 64, 64, 3, 3, 1, 1, 1, 2, 4, 64),
    ConvShape("win_3x3_28", 2, 28, 28, 128, 128, 3, 3, 1, 1, 1, 2, 4, 64),
    ConvShape("win_3x3_14", 3, 14, 14, 64, 96, 3, 3, 1, 1, 1, 2, 4, 32),              # row blocks of 8 and 6 rows
    ConvShape("win_5x5_dil2", 1, 20, 20, 32, 32, 5, 5, 1, 4, 2, 2, 4, 16),
    ConvShape("win_nopad", 1, 18, 18, 32, 64, 3, 3, 1, 0, 1, 1, 4, 64),
    ConvShape("win_wide_122", 1, 6, 120, 32, 32, 3, 3, 1, 1, 1, 2, 4, 32),            # one output row per M-tile
    ConvShape("win_wide_132", 1, 6, 130, 32, 32, 3, 3, 1, 1, 1, 2, 4, 32),            # an output row spans two M-tiles
    ConvShape("win_7x7_map", 4, 7, 7, 64, 64, 3, 3, 1, 1, 1, 2, 4, 64),
    ConvShape("win_many_items", 6, 56, 56, 32, 64, 3, 3, 1, 1, 1, 2, 4, 32),          # 168+ work items: several per CTA
]


@pytest.mark.parametrize("s", WINDOW, ids=lambda s: s.name)
def test_window_shapes(nm, s):
    _run(nm, s, need_variant=[6])


@pytest.mark.parametrize("s", WINDOW[:5] + WINDOW[6:7], ids=lambda s: s.name)
def test_window_shapes_integer_exact(nm, s):
    _run(nm, s, integer=True, need_variant=[6])


# pointwise layers whose channel counts are not multiples of 32 (MobileNet-like): the expanded-operand kernel lets
# the TMA unit zero-fill the last input block and pads the weight rows
POINTWISE = [
    ConvShape("pw_cin24", 2, 56, 56, 24, 144, 1, 1, 1, 0, 1, 2, 4, 16),
    ConvShape("pw_cout24", 2, 56, 56, 96, 24, 1, 1, 1, 0, 1, 2, 4, 8),
    ConvShape("pw_cin144_cout24", 2, 40, 40, 144, 24, 1, 1, 1, 0, 1, 2, 4, 8),
    ConvShape("pw_cin16_cout96", 1, 112, 112, 16, 96, 1, 1, 1, 0, 1, 2, 4, 16),
    ConvShape("pw_cout16", 1, 112, 112, 32, 16, 1, 1, 1, 0, 1, 2, 4, 16),
    ConvShape("pw_cout40_stride2", 2, 57, 57, 48, 40, 1, 1, 2, 0, 1, 1, 4, 8),       # strided, ragged pixel tail (841 pixels)
]


@pytest.mark.parametrize("s", POINTWISE, ids=lambda s: s.name)
def test_pointwise_ragged_channels(nm, s):
    _run(nm, s, need_variant=[1, 4])


@pytest.mark.parametrize("s", POINTWISE, ids=lambda s: s.name)
def test_pointwise_ragged_channels_integer_exact(nm, s):
    _run(nm, s, integer=True, need_variant=[4])


# pair kernel (variant 7): clusters of two CTAs share one 256-pixel x bn MMA
PAIR = [
    ConvShape("pair_one", 1, 16, 16, 128, 256, 3, 3, 1, 1, 1, 2, 4, 64),              # 2 pixel blocks: one pair, one item
    ConvShape("pair_odd_blocks", 2, 13, 13, 128, 256, 3, 3, 1, 1, 1, 2, 4, 64),       # 338 pixels: 3 blocks, the 4th is empty
    ConvShape("pair_1x1_long_k", 2, 14, 14, 1024, 128, 1, 1, 1, 0, 1, 2, 4, 64),      # 32 stages: the ring wraps
    ConvShape("pair_stride2", 2, 29, 29, 64, 128, 3, 3, 2, 1, 1, 1, 4, 32),
    ConvShape("pair_many_items", 8, 56, 56, 32, 256, 3, 3, 1, 1, 1, 2, 4, 64),        # 98 block pairs x 1-2 slices: several items per pair
]


@pytest.mark.parametrize("s", PAIR, ids=lambda s: s.name)
def test_pair_shapes(nm, s):
    _run(nm, s, need_variant=[4, 7])


@pytest.mark.parametrize("s", PAIR[:4], ids=lambda s: s.name)
def test_pair_shapes_integer_exact(nm, s):
    _run(nm, s, integer=True, need_variant=[7])


@pytest.mark.parametrize("s", MEDIUM, ids=lambda s: s.name)
def test_medium_shapes(nm, s):
    # the stream kernel takes tiles that are multiples of 16 channels and its seven N:M patterns
    # on inputs of at least 128 KiB
    stream = (s.tile_t % 16 == 0 and s.c_out % 32 == 0 and s.batch * s.h * s.w * s.c_in * 4 >= 131072 and
              (s.n_keep, s.m_group) in ((1, 4), (2, 4), (3, 4), (4, 4), (1, 8), (2, 8), (4, 8)))
    big = s.batch * s.h * s.w * s.c_in * 4 >= 131072
    expand = big and s.c_in % 32 == 0 and s.c_out % 32 == 0     # any tile width, any N:M
    _run(nm, s, need_variant=[3 if stream else 2] + ([4] if expand else []))


@pytest.mark.parametrize("s", MEDIUM[:6] + MEDIUM[13:], ids=lambda s: s.name)
def test_medium_shapes_integer_exact(nm, s):
    _run(nm, s, integer=True)


def test_asymmetric_geometry(nm):
    """3x5 kernel, stride (1, 2), padding (1, 2), dilation (2, 1): catches any h / w mix-up."""
    import oracle
    g = torch.Generator().manual_seed(77)
    w = torch.randint(-3, 4, (32, 3, 5, 64), generator=g).float()
    x = torch.randint(-3, 4, (2, 18, 22, 64), generator=g).float()
    b = torch.randint(-3, 4, (32,), generator=g).float()
    stride, pad, dil = (1, 2), (1, 2), (2, 1)
    vr, ir = oracle.prune(w.numpy(), 2, 4, 16)
    yr = oracle.conv2d(vr, ir, 3, 5, 64, 16, x.numpy(), stride, pad, dil, b.numpy(), True)
    hnd = nm.nm_prune(w.cuda(), 2, 4, 16)
    for plan in _plans(nm, None):
        try:
            y = nm.nm_conv2d(hnd, x.cuda(), 3, 5, stride, pad, dil, b.cuda(), True, plan=plan)
        except nm.NmError as e:
            if plan is not None and e.status == nm.NM_ERR_UNSUPPORTED:
                continue
            raise
        nm.nm_weights_check(hnd)
        torch.cuda.synchronize()
        assert np.array_equal(y.cpu().numpy(), yr), f"plan {plan.as_dict() if plan else None}"


@pytest.mark.parametrize("s", SMALL[:8], ids=lambda s: s.name)
def test_small_shapes_integer_exact(nm, s):
    _run(nm, s, integer=True)


@pytest.mark.parametrize("integer", [False, True], ids=["normal", "integer_exact"])
def test_split_k_plans(nm, integer):
    """Few pixel blocks and a long reduction axis: the expanded-operand kernel with the axis split over
    2, 3 and 4 CTAs (partial sums through the handle's scratch, reserved by nm_autotune, then reduced)."""
    s = ConvShape("splitk_3x3", 2, 14, 14, 256, 64, 3, 3, 1, 1, 1, 2, 4, 32)        # K = 2304: 72 blocks of 32
    w, x, b = tensors_for(s, integer)
    vr, ir, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd = x.cuda(), b.cuda()
    plan = nm.nm_plan_t()
    plan.variant, plan.bn, plan.split = 4, 64, 2
    with pytest.raises(nm.NmError) as e:                      # no scratch yet: the plan is refused
        nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    need = nm.nm_plan_scratch_bytes(hnd, xd.shape, s.stride, s.pad, s.dil, plan)
    assert need == 2 * 512 * 64 * 4                           # splits x pixels padded to 128 x channels x 4 bytes
    nm.nm_weights_reserve(hnd, need)                          # explicit reservation: now the plan runs
    y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
    torch.cuda.synchronize()
    assert_conv_close(y.cpu().numpy(), yr)
    best, ms = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)   # reserves for 4 splits
    assert ms > 0
    for splits in (2, 3, 4):
        for bn in (32, 64):
            plan = nm.nm_plan_t()
            plan.variant, plan.bn, plan.split = 4, bn, splits
            plan.kblk = 2 if bn == 64 else 0                  # K / 32 / splits = 36, 24, 18: two blocks per stage fit
            plan.issuers = 2 if splits == 3 else 0            # one of the splits with two issuer threads
            for _ in range(2):                                # twice: the scratch is reused
                y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
            nm.nm_weights_check(hnd)
            torch.cuda.synchronize()
            if integer:
                assert np.array_equal(y.cpu().numpy(), yr), (splits, bn)
            else:
                assert_conv_close(y.cpu().numpy(), yr)
    y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=best)
    torch.cuda.synchronize()
    if not integer:
        assert_conv_close(y.cpu().numpy(), yr)


BALANCED = [
    ConvShape("bal_few_items", 2, 14, 14, 256, 64, 3, 3, 1, 1, 1, 2, 4, 32),          # 4 items of 72 stages over all SMs: ~37 CTAs per item
    ConvShape("bal_many_items", 8, 56, 56, 32, 256, 3, 3, 1, 1, 1, 2, 4, 64),         # 392 items of 9 stages: whole items and parts per CTA
    ConvShape("bal_1x1_ragged", 3, 13, 13, 1024, 128, 1, 1, 1, 0, 1, 2, 4, 64),       # 507 pixels: ragged last block, 32 stages
]


@pytest.mark.parametrize("integer", [False, True], ids=["normal", "integer"])
@pytest.mark.parametrize("s", BALANCED, ids=lambda s: s.name)
def test_balanced_plans(nm, s, integer):
    """Expanded-operand kernel with the (item, stage) pairs of the layer cut into one equal range per SM
    (plan.split = -1): CTAs that share an item exchange partial sums through the handle's scratch."""
    w, x, b = tensors_for(s, integer)
    vr, ir, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd = x.cuda(), b.cuda()
    ran = 0
    for bn, kblk, stages, issuers in ((64, 0, 0, 0), (128, 2, 0, 0), (32, 1, 2, 0), (256, 0, 0, 0), (256, 0, 0, 2), (128, 2, 0, 2), (64, 1, 2, 2)):
        if s.c_out % bn:
            continue
        plan = nm.nm_plan_t()
        plan.variant, plan.bn, plan.split, plan.kblk, plan.stages, plan.issuers = 4, bn, -1, kblk, stages, issuers
        need = nm.nm_plan_scratch_bytes(hnd, xd.shape, s.stride, s.pad, s.dil, plan)
        assert need >= 128 * bn * 4
        nm.nm_weights_reserve(hnd, need)
        try:
            for _ in range(3):                                # several launches: slots and flags are reused
                y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
        except nm.NmError as e:
            if e.status == nm.NM_ERR_UNSUPPORTED:
                continue                                      # e.g. K / 32 odd with two blocks per stage
            raise
        nm.nm_weights_check(hnd)
        torch.cuda.synchronize()
        ran += 1
        if integer:
            assert np.array_equal(y.cpu().numpy(), yr), (s.name, bn)
        else:
            assert_conv_close(y.cpu().numpy(), yr)
    assert ran >= 2


# Groups as wide as the input-channel axis (the paper's adaptive setting, Sec. 3.1: M may span all input
# channels, N = (1 - sparsity) * M): every kernel that reads the tap table or the expanded weights takes them.
LARGE_M = [
    ConvShape("m_is_cin_1x1", 2, 14, 14, 256, 128, 1, 1, 1, 0, 1, 64, 256, 32),       # 75 % sparsity, M = C_in
    ConvShape("m_is_cin_3x3", 1, 16, 16, 128, 64, 3, 3, 1, 1, 1, 64, 128, 8),         # 50 %, M = C_in, tile 8
    ConvShape("m_is_row", 1, 12, 12, 64, 64, 3, 3, 1, 1, 1, 144, 576, 16),            # 75 %, M = the whole row K
    ConvShape("m_64_of_96", 2, 10, 10, 96, 32, 1, 1, 1, 0, 1, 24, 96, 32),
]


@pytest.mark.parametrize("s", LARGE_M, ids=lambda s: s.name)
def test_large_groups(nm, s):
    big = s.batch * s.h * s.w * s.c_in * 4 >= 131072
    _run(nm, s, need_variant=[1] + ([4] if big else []))


@pytest.mark.parametrize("s", LARGE_M[:2], ids=lambda s: s.name)
def test_large_groups_integer_exact(nm, s):
    _run(nm, s, integer=True)


def test_no_bias_no_relu(nm):
    _run(nm, SMALL[0].with_(relu=False), use_bias=False)


@pytest.mark.parametrize("s", inputs.config_resnet3x3(), ids=lambda s: s.name)
def test_resnet3x3_full_layer(nm, s):
    _run(nm, s)


@pytest.mark.parametrize("s", [c.with_(batch=8) for c in inputs.config_bottleneck1x1()], ids=lambda s: s.name)
def test_bottleneck1x1_batch8(nm, s):
    _run(nm, s)


def test_argument_errors(nm):
    s = inputs.config_tiny()
    w, x, b = tensors_for(s)
    hnd = nm.nm_prune(w.cuda(), 2, 4, 8)
    xd = x.cuda()
    with pytest.raises(nm.NmError) as e:
        nm.nm_conv2d(hnd, xd, 3, 3, 0, 1, 1)              # stride 0
    assert e.value.status == nm.NM_ERR_INVALID_ARG
    with pytest.raises(nm.NmError) as e:
        nm.nm_conv2d(hnd, xd[:, :2, :2].contiguous(), 3, 3, 1, 0, 1)   # kernel larger than the image
    assert e.value.status == nm.NM_ERR_INVALID_ARG
    bad = torch.zeros(xd.numel() + 1, device="cuda")[1:].view_as(xd)   # 4-byte aligned only
    with pytest.raises(nm.NmError) as e:
        nm.nm_conv2d(hnd, bad, 3, 3, 1, 1, 1)
    assert e.value.status == nm.NM_ERR_INVALID_ARG
    plan = nm.nm_plan_t()
    plan.variant = 99
    with pytest.raises(nm.NmError) as e:
        nm.nm_conv2d(hnd, xd, 3, 3, 1, 1, 1, plan=plan)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    # the context is still usable afterwards
    y = nm.nm_conv2d(hnd, xd, 3, 3, 1, 1, 1)
    torch.cuda.synchronize()
    assert torch.isfinite(y).all()


def test_expired_wait_is_reported_and_the_context_survives(nm):
    """A device-side wait that runs out (on a barrier nothing completes) ends its kernel normally, is
    reported once through the status word, and leaves the handle and the context usable."""
    s = inputs.config_tiny()
    w, x, b = tensors_for(s)
    _, _, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    nm.nm_weights_check(hnd)                                   # clean to begin with
    nm.nm_selftest_wait_expiry(hnd)
    with pytest.raises(nm.NmError) as e:
        nm.nm_weights_check(hnd)
    assert e.value.status == nm.NM_ERR_TIMEOUT
    nm.nm_weights_check(hnd)                                   # reported once, then cleared
    y = nm.nm_conv2d(hnd, x.cuda(), s.kh, s.kw, s.stride, s.pad, s.dil, b.cuda(), s.relu)
    nm.nm_weights_check(hnd)
    torch.cuda.synchronize()
    assert_conv_close(y.cpu().numpy(), yr)


def test_host_buffer_entry_point(nm):
    s = inputs.config_tiny()
    w, x, b = tensors_for(s)
    _, _, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xh, bh = x.pin_memory(), b.pin_memory()
    yh = torch.empty(yr.shape, dtype=torch.float32).pin_memory()
    xd, bd, yd = torch.empty_like(x, device="cuda"), torch.empty_like(b, device="cuda"), torch.empty(yr.shape, device="cuda")
    nm.nm_conv2d_host(hnd, xh, xd, s.stride, s.pad, s.dil, bh, bd, s.relu, yh, yd)
    torch.cuda.synchronize()
    assert_conv_close(yh.numpy(), yr)


def test_autotune_returns_a_working_plan(nm):
    s = SMALL[1]
    w, x, b = tensors_for(s)
    _, _, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    plan, ms = nm.nm_autotune(hnd, x.cuda(), s.stride, s.pad, s.dil, b.cuda(), s.relu, kh=s.kh, kw=s.kw)
    assert plan.variant >= 1 and ms > 0
    y = nm.nm_conv2d(hnd, x.cuda(), s.kh, s.kw, s.stride, s.pad, s.dil, b.cuda(), s.relu, plan=plan)
    torch.cuda.synchronize()
    assert_conv_close(y.cpu().numpy(), yr)
    tile, plan, ms = nm.nm_autotune_tile(w.cuda(), s.n_keep, s.m_group, [16, 32], x.cuda(), s.stride, s.pad, s.dil,
                                         b.cuda(), s.relu)
    assert tile in (16, 32) and ms > 0


def test_autotune_uses_the_plan_cache(nm, tmp_path, monkeypatch):
    """With NM_PLAN_CACHE set, nm_autotune stores what it found and the next call on the same layer returns that
    plan without tuning; a cached plan the layer does not admit is ignored and replaced."""
    s = ConvShape("cache_3x3", 2, 16, 16, 64, 64, 3, 3, 1, 1, 1, 2, 4, 32)
    w, x, b = tensors_for(s)
    vr, ir, yr = oracle_layer(s, w, x, b)
    path = str(tmp_path / "plans.txt")
    monkeypatch.setenv("NM_PLAN_CACHE", path)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd = x.cuda(), b.cuda()
    plan1, ms1 = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)
    key = nm.nm_plan_key(s.c_out, s.kh, s.kw, s.c_in, s.n_keep, s.m_group, s.tile_t, xd.shape, s.stride, s.pad, s.dil, True, s.relu)
    assert nm.nm_plan_cache_lookup(path, key).as_dict() == plan1.as_dict()
    forced = nm.nm_plan_t()
    forced.variant = 1                                  # the slowest kernel: tuning would never pick it here
    nm.nm_plan_cache_store(path, key, forced)
    plan2, ms2 = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)
    assert plan2.variant == 1 and ms2 > 0
    y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan2)
    torch.cuda.synchronize()
    assert_conv_close(y.cpu().numpy(), yr)
    bad = nm.nm_plan_t()
    bad.variant, bad.bn = 4, 96                         # 96 channels per CTA do not divide 64: not admissible
    nm.nm_plan_cache_store(path, key, bad)
    plan3, _ = nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)
    assert plan3.as_dict() != bad.as_dict()
    assert nm.nm_plan_cache_lookup(path, key).as_dict() == plan3.as_dict()


def test_balanced_plan_beside_a_busy_stream(nm):
    """A balanced plan's CTAs wait (with a bound) for flags raised by other CTAs of the same launch, which assumes
    that all of them are resident.  With another stream keeping SMs busy the launch must still either finish with
    the right result or report NM_ERR_TIMEOUT through the status word: never hang, never return wrong numbers."""
    s = BALANCED[0]
    w, x, b = tensors_for(s, True)
    vr, ir, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    other = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd = x.cuda(), b.cuda()
    plan = nm.nm_plan_t()
    plan.variant, plan.bn, plan.split = 4, 64, -1
    nm.nm_weights_reserve(hnd, nm.nm_plan_scratch_bytes(hnd, xd.shape, s.stride, s.pad, s.dil, plan))
    busy = torch.cuda.Stream()
    y_other = torch.empty((s.batch, s.ho, s.wo, s.c_out), device="cuda")
    torch.cuda.synchronize()
    outcomes = set()
    for _ in range(5):
        with torch.cuda.stream(busy):                   # a queue of persistent kernels on the other stream
            for _k in range(20):
                nm.nm_conv2d(other, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, y=y_other)
        y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)
        try:
            nm.nm_weights_check(hnd)
            torch.cuda.synchronize()
            assert np.array_equal(y.cpu().numpy(), yr)
            outcomes.add("ok")
        except nm.NmError as e:
            assert e.status == nm.NM_ERR_TIMEOUT
            outcomes.add("timeout")
        torch.cuda.synchronize()
    assert outcomes <= {"ok", "timeout"} and outcomes
    nm.nm_weights_check(other)
    y = nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, plan=plan)   # alone again: must be right
    nm.nm_weights_check(hnd)
    torch.cuda.synchronize()
    assert np.array_equal(y.cpu().numpy(), yr)
