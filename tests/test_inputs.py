"""The seeded input recipes are deterministic and have the stated shapes / sizes."""
import torch

from paper_2507_17301_b200 import inputs


def test_seeded_draws_repeat():
    s = inputs.config_tiny()
    assert torch.equal(inputs.make_weights(s), inputs.make_weights(s))
    assert torch.equal(inputs.make_activations(s), inputs.make_activations(s))
    assert not torch.equal(inputs.make_weights(s, 1), inputs.make_weights(s, 0))
    assert inputs.make_weights(s).shape == (32, 3, 3, 16)
    assert inputs.make_activations(s).shape == (1, 14, 14, 16)
    assert (s.k, s.kk, s.pixels, s.ho, s.wo) == (144, 72, 196, 14, 14)


def test_kaiming_scale():
    s = inputs.config_resnet3x3()[0]
    w = inputs.make_weights(s)
    assert abs(float(w.std()) - (2.0 / s.k) ** 0.5) < 0.02 * (2.0 / s.k) ** 0.5


def test_resnet_stacks_have_the_published_conv_counts_and_flops():
    r50 = inputs.resnet_conv_stack(50, 64, 2, 4)
    assert len(r50) == 53
    dense = sum(2 * s.pixels * s.c_out * s.k for s in r50) / 64
    assert abs(dense / 1e9 - 8.17) < 0.1  # ~4.1 GMAC per image
    r101 = inputs.resnet_conv_stack(101, 128, 1, 4)
    assert len(r101) == 104
    assert r50[0].kk == r50[0].k == 147  # stem keeps every column
    # spatial sizes chain: last block works on 7x7
    assert (r50[-1].ho, r50[-1].c_out) == (7, 2048)
    # basic-block networks: 1 + 16 + 3 = 20 and 1 + 32 + 3 = 36 convolutions, ~1.8 and ~3.6 GMAC per image
    r18, r34 = inputs.resnet_conv_stack(18, 1, 2, 4), inputs.resnet_conv_stack(34, 1, 2, 4)
    assert (len(r18), len(r34)) == (20, 36)
    assert abs(sum(s.pixels * s.c_out * s.k for s in r18) / 1e9 - 1.81) < 0.05
    assert abs(sum(s.pixels * s.c_out * s.k for s in r34) / 1e9 - 3.66) < 0.05
    assert (r34[-1].ho, r34[-1].c_out, r34[-1].kh) == (7, 512, 3)


def test_mobilenet_v2_pointwise_shapes():
    layers = inputs.mobilenet_v2_pointwise(1, 2, 4)
    assert len(layers) == 34                                   # 16 expansions + 17 projections + the last 1x1
    assert all(s.kh == 1 and s.kw == 1 and s.stride == 1 for s in layers)
    assert (layers[0].c_in, layers[0].c_out, layers[0].h) == (32, 16, 112)
    assert (layers[-1].c_in, layers[-1].c_out, layers[-1].h) == (320, 1280, 7)
    # a projection's input is its block's expansion output; the chain of block outputs is 16, 24, ..., 320
    outs = [s.c_out for s in layers if s.name.endswith("_project")]
    assert outs == [16, 24, 24, 32, 32, 32, 64, 64, 64, 64, 96, 96, 96, 160, 160, 160, 320]
    for a, b in zip(layers, layers[1:]):
        if a.name.endswith("_expand"):
            assert b.name.endswith("_project") and b.c_in == a.c_out == 6 * a.c_in
    # multiply-accumulates of the dense pointwise layers at 224 x 224 (a check of the map sizes)
    macs = sum(s.ho * s.wo * s.c_in * s.c_out for s in layers)
    assert 250e6 < macs < 300e6



def test_bench_host_logic(tmp_path, monkeypatch):
    """bench.py's workload selection, algorithmic bytes and the look-up of recorded DRAM traffic (no GPU)."""
    import bench

    monkeypatch.setitem(bench.WORKLOAD, "net", "resnet")
    r50 = bench.workload(64)
    assert len(r50) == 53 and bench.workload_name(64) == "resnet50_conv_stack_b64_224_2of4"
    stem = r50[0]
    # stem: input 64 x 224 x 224 x 3, output 64 x 112 x 112 x 64, all 64 x 147 weights kept, one tile's indices, bias
    assert bench.algorithmic_bytes(stem) == 4 * (64 * 224 * 224 * 3 + 64 * 112 * 112 * 64 + 64 * 147 + 64) + 2 * 147
    assert bench.useful_flops(stem) == 2 * 64 * 112 * 112 * 64 * 147
    monkeypatch.setitem(bench.WORKLOAD, "net", "mobilenet_v2")
    assert len(bench.workload(8)) == 34 and bench.workload_name(8).startswith("mobilenet_v2_pointwise")
    monkeypatch.setitem(bench.WORKLOAD, "net", "resnet")
    # a traffic summary counts only while the kernel source it was taken from is unchanged
    got = bench.recorded_traffic("k_conv_expand")
    if got is not None:
        assert 0.3 < got < 1.5          # DRAM bytes per algorithmic byte: no re-reads, some output still in L2
    monkeypatch.setattr(bench, "source_digest", lambda kernel: "0" * 16)
    assert bench.recorded_traffic("k_conv_expand") is None
    assert bench.recorded_traffic("k_no_such_kernel") is None
