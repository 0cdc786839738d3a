"""Seeded synthetic inputs and workload shapes (no arithmetic of the method lives here).

Both the CPU oracle's tests and the CUDA path's tests / benchmark draw their tensors
from this module, so that the two sides see bit-identical inputs.  It holds only
random-number recipes and layer-shape tables: activations ~ N(0, 1); weights either
N(0, 1) or "Kaiming-normal" N(0, 2 / K) with K = kh * kw * c_in (fan-in); bias N(0, 1).
Seeds: weights 0, activations 1, bias 2, each plus the layer's index in a stack.

The shapes are those of the workloads the paper evaluates (torchvision ResNets,
Sec. 4.1.2); its ImageNet images and retrained weights are replaced by these draws.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import torch


@dataclass(frozen=True)
class ConvShape:
    """One convolution layer: NHWC input ``[batch, h, w, c_in]``, OHWI weights ``[c_out, kh, kw, c_in]``."""

    name: str
    batch: int
    h: int
    w: int
    c_in: int
    c_out: int
    kh: int = 1
    kw: int = 1
    stride: int = 1
    pad: int = 0
    dil: int = 1
    n_keep: int = 2
    m_group: int = 4
    tile_t: int = 64
    relu: bool = True
    kaiming: bool = True
    count: int = 1  # how many layers of a network share this exact shape

    @property
    def k(self) -> int:
        return self.kh * self.kw * self.c_in

    @property
    def ho(self) -> int:
        return (self.h + 2 * self.pad - self.dil * (self.kh - 1) - 1) // self.stride + 1

    @property
    def wo(self) -> int:
        return (self.w + 2 * self.pad - self.dil * (self.kw - 1) - 1) // self.stride + 1

    @property
    def pixels(self) -> int:
        return self.batch * self.ho * self.wo

    @property
    def kk(self) -> int:
        full, tail = divmod(self.k, self.m_group)
        return full * self.n_keep + min(tail, self.n_keep)

    def with_(self, **kw) -> "ConvShape":
        return replace(self, **kw)


def _normal(shape, seed: int, std: float = 1.0) -> torch.Tensor:
    g = torch.Generator(device="cpu")
    g.manual_seed(seed)
    return torch.randn(shape, generator=g, dtype=torch.float32) * std


def make_weights(s: ConvShape, layer: int = 0) -> torch.Tensor:
    """Dense OHWI fp32 weights: N(0, 2/K) if ``s.kaiming`` else N(0, 1); seed 0 + layer."""
    std = (2.0 / s.k) ** 0.5 if s.kaiming else 1.0
    return _normal((s.c_out, s.kh, s.kw, s.c_in), 0 + 1000 * layer, std)


def make_activations(s: ConvShape, layer: int = 0, batch: int | None = None) -> torch.Tensor:
    """NHWC fp32 activations ~ N(0, 1); seed 1 + layer."""
    return _normal((s.batch if batch is None else batch, s.h, s.w, s.c_in), 1 + 1000 * layer)


def make_bias(s: ConvShape, layer: int = 0) -> torch.Tensor:
    """Bias ~ N(0, 1) (stands for a folded batch-norm shift); seed 2 + layer."""
    return _normal((s.c_out,), 2 + 1000 * layer)


def make_int_case(s: ConvShape, layer: int = 0):
    """Small-integer weights, activations and bias in {-4..4}: every product and partial sum
    is exactly representable in TF32 / fp32, so any correct implementation agrees exactly."""
    g = torch.Generator(device="cpu")
    g.manual_seed(7 + 1000 * layer)
    w = torch.randint(-4, 5, (s.c_out, s.kh, s.kw, s.c_in), generator=g).float()
    x = torch.randint(-4, 5, (s.batch, s.h, s.w, s.c_in), generator=g).float()
    b = torch.randint(-4, 5, (s.c_out,), generator=g).float()
    return w, x, b


# ---------------------------------------------------------------------------------------------
# Named configurations
# ---------------------------------------------------------------------------------------------

def config_tiny() -> ConvShape:
    """Single 3x3 conv, batch 1, 14x14, 16 -> 32, 2:4, tile 8, N(0,1) weights, bias, ReLU."""
    return ConvShape("tiny3x3", 1, 14, 14, 16, 32, 3, 3, 1, 1, 1, 2, 4, 8, True, False)


def config_resnet3x3():
    """ResNet-style 3x3 layer, batch 32, 14x14, 256 -> 256; {2:4, 1:4, 2:8} x tile {32, 64}."""
    out = []
    for (n, m) in ((2, 4), (1, 4), (2, 8)):
        for t in (32, 64):
            out.append(ConvShape(f"c3x3_256_{n}of{m}_T{t}", 32, 14, 14, 256, 256, 3, 3, 1, 1, 1, n, m, t))
    return out


def config_bottleneck1x1():
    """1x1 bottleneck convs (pure sparse GEMM): batch 64; 2:4 and 1:8."""
    out = []
    for (n, m) in ((2, 4), (1, 8)):
        out.append(ConvShape(f"c1x1_1024_256_{n}of{m}", 64, 14, 14, 1024, 256, n_keep=n, m_group=m))
        out.append(ConvShape(f"c1x1_256_1024_{n}of{m}", 64, 14, 14, 256, 1024, n_keep=n, m_group=m))
        out.append(ConvShape(f"c1x1_512_128_{n}of{m}", 64, 28, 28, 512, 128, n_keep=n, m_group=m))
    return out


def _basic_block_stack(depth: int, batch: int, n_keep: int, m_group: int, tile_t: int, image: int):
    """ResNet-18 / 34 (He et al. 2016): 7x7/2 stem, 3x3/2 max-pool, four stages of basic blocks (two
    3x3 convolutions; the first one of a stage's first block has stride 2 from stage 2 on, with a
    1x1/2 projection on its shortcut).  The networks on which the paper reports its largest gains."""
    blocks = {18: (2, 2, 2, 2), 34: (3, 4, 6, 3)}[depth]
    layers = [ConvShape("stem7x7", batch, image, image, 3, 64, 7, 7, 2, 3, 1, 1, 1, min(tile_t, 64))]
    hw = (layers[0].ho + 2 - 3) // 2 + 1   # max-pool -> 56
    c_prev = 64
    for si, nb in enumerate(blocks):
        width = 64 << si
        for bi in range(nb):
            stride = 2 if (bi == 0 and si > 0) else 1
            pre = f"s{si + 1}b{bi + 1}"
            mk = dict(n_keep=n_keep, m_group=m_group, tile_t=tile_t)
            layers.append(ConvShape(pre + "_c1", batch, hw, hw, c_prev, width, 3, 3, stride, 1, **mk))
            hw_out = (hw + 2 - 3) // stride + 1
            layers.append(ConvShape(pre + "_c2", batch, hw_out, hw_out, width, width, 3, 3, 1, 1, relu=False, **mk))
            if stride == 2:
                layers.append(ConvShape(pre + "_ds", batch, hw, hw, c_prev, width, 1, 1, 2, 0, relu=False, **mk))
            hw = hw_out
            c_prev = width
    return layers


def resnet_conv_stack(depth: int, batch: int, n_keep: int, m_group: int, tile_t: int = 64, image: int = 224):
    """Every convolution of a ResNet in network order: bottleneck ResNets (50 / 101 / 152) as described
    below, basic-block ResNets (18 / 34) through ``_basic_block_stack``.

    Standard architecture (He et al. 2016): 7x7/2 stem, 3x3/2 max-pool, four stages of
    bottleneck blocks (1x1, 3x3, 1x1; the stride sits on the 3x3 of a stage's first block;
    a 1x1 projection on the first block's shortcut).  The stem keeps every column
    (Sec. 4.1.2: the first convolution is not pruned): it is returned with N = M = 1.
    """
    if depth in (18, 34):
        return _basic_block_stack(depth, batch, n_keep, m_group, tile_t, image)
    blocks = {50: (3, 4, 6, 3), 101: (3, 4, 23, 3), 152: (3, 8, 36, 3)}[depth]
    layers = [ConvShape("stem7x7", batch, image, image, 3, 64, 7, 7, 2, 3, 1, 1, 1, min(tile_t, 64))]
    hw = layers[0].ho  # 112
    hw = (hw + 2 - 3) // 2 + 1  # 3x3/2 max-pool, pad 1 -> 56
    c_prev = 64
    for si, nb in enumerate(blocks):
        width = 64 << si
        for bi in range(nb):
            stride = 2 if (bi == 0 and si > 0) else 1
            pre = f"s{si + 1}b{bi + 1}"
            mk = dict(n_keep=n_keep, m_group=m_group, tile_t=tile_t)
            layers.append(ConvShape(pre + "_c1", batch, hw, hw, c_prev, width, **mk))
            layers.append(ConvShape(pre + "_c2", batch, hw, hw, width, width, 3, 3, stride, 1, **mk))
            hw_out = (hw + 2 - 3) // stride + 1
            # no ReLU straight after the third conv or the projection: the residual sum comes first
            layers.append(ConvShape(pre + "_c3", batch, hw_out, hw_out, width, 4 * width, relu=False, **mk))
            if bi == 0:
                layers.append(ConvShape(pre + "_ds", batch, hw, hw, c_prev, 4 * width, 1, 1, stride, 0,
                                        relu=False, **mk))
            hw = hw_out
            c_prev = 4 * width
    return layers


def mobilenet_v2_pointwise(batch: int, n_keep: int, m_group: int, tile_t: int = 16, image: int = 224):
    """The pointwise (1x1) convolutions of MobileNet-V2 in network order: per inverted-residual block the
    expansion (absent where the expansion factor is 1) and the linear projection, then the final 1x1
    convolution.  These are the layers the paper prunes in this network (Sec. 4.5: the depthwise
    convolutions stay dense and are not part of the pruned path), so the 3x3 stem and the depthwise
    layers only appear here through the map sizes they produce.

    Standard architecture (Sandler et al. 2018): stem 3x3/2 to 32 channels, blocks given as
    (expansion t, channels c, repeats n, stride s), the stride on the first repeat's depthwise layer.
    Several channel counts (16, 24, 144, ...) are not multiples of 32: those layers exercise the general kernels.
    """
    table = ((1, 16, 1, 1), (6, 24, 2, 2), (6, 32, 3, 2), (6, 64, 4, 2), (6, 96, 3, 1), (6, 160, 3, 2), (6, 320, 1, 1))
    mk = dict(n_keep=n_keep, m_group=m_group, tile_t=tile_t)
    layers = []
    hw = (image + 2 - 3) // 2 + 1   # after the stem: 112
    c_prev = 32
    for bi, (t, c, n, s) in enumerate(table):
        for ri in range(n):
            stride = s if ri == 0 else 1
            pre = f"b{bi + 1}r{ri + 1}"
            hidden = c_prev * t
            if t != 1:
                layers.append(ConvShape(pre + "_expand", batch, hw, hw, c_prev, hidden, **mk))      # followed by ReLU6 in the network; ReLU here
            hw = (hw + 2 - 3) // stride + 1                                                            # the depthwise 3x3 in between
            layers.append(ConvShape(pre + "_project", batch, hw, hw, hidden, c, relu=False, **mk))   # linear bottleneck
            c_prev = c
    layers.append(ConvShape("last_1x1", batch, hw, hw, c_prev, 1280, **mk))
    return layers

