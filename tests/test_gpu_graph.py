"""Launches recorded in a CUDA graph and replayed give the result of direct launches, for every kind of
plan that keeps state between kernels: split-K (partial sums + reduction pass) and balanced ranges (per-SM
slots and flags that their readers lower again, so a recorded launch can be replayed any number of times)."""
import numpy as np
import pytest
import torch

from paper_2507_17301_b200.inputs import ConvShape
from parity import assert_conv_close, oracle_layer, tensors_for

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


def _plan(nm, **kw):
    p = nm.nm_plan_t()
    for k, v in kw.items():
        setattr(p, k, v)
    return p


def test_replayed_graph_matches_direct_launches(nm):
    s = ConvShape("graph_3x3", 2, 14, 14, 256, 64, 3, 3, 1, 1, 1, 2, 4, 32)          # K = 2304: 4 items of 72 stages
    w, x, b = tensors_for(s, True)                                                    # integer-valued: exact sums
    _, _, yr = oracle_layer(s, w, x, b)
    hnd = nm.nm_prune(w.cuda(), s.n_keep, s.m_group, s.tile_t)
    xd, bd = x.cuda(), b.cuda()
    nm.nm_autotune(hnd, xd, s.stride, s.pad, s.dil, bd, s.relu, kh=s.kh, kw=s.kw)    # reserves the scratch
    plans = [None, _plan(nm, variant=4, bn=64), _plan(nm, variant=4, bn=64, split=3), _plan(nm, variant=4, bn=64, split=-1),
             _plan(nm, variant=4, bn=32, split=-1, kblk=2), _plan(nm, variant=6, bn=64, split=1)]
    outs = [torch.empty((s.batch, s.ho, s.wo, s.c_out), device="cuda") for _ in plans]

    def launch_all():
        for plan, y in zip(plans, outs):
            nm.nm_conv2d(hnd, xd, s.kh, s.kw, s.stride, s.pad, s.dil, bd, s.relu, y=y, plan=plan)

    launch_all()                                                                      # warm-up outside the capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            launch_all()
    torch.cuda.current_stream().wait_stream(side)
    for rep in range(3):
        for y in outs:
            y.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        nm.nm_weights_check(hnd)
        for plan, y in zip(plans, outs):
            assert np.array_equal(y.cpu().numpy(), yr), (rep, plan.as_dict() if plan else None)
    # and the handle still serves direct launches afterwards
    launch_all()
    torch.cuda.synchronize()
    assert_conv_close(outs[3].cpu().numpy(), yr)
