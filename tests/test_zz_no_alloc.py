"""The allocation-free pruning entry point (nm_prune_noalloc) against the regular one and the CPU oracle.

Collected last on purpose: a run that stops at the first failure has then already run every other
test.  The entry point exists for callers that cannot allocate device memory themselves (a plug-in
inside a server that has reserved all of HBM, a loop that cannot take cudaMalloc's device-wide
synchronisation); it keeps its scratch in one array built into the library, which every call shares
and which keeps whatever the previous call left there.  So the check is made on two calls in a
row with different problems, the second smaller than the first, and each must reproduce nm_prune's
canonical output bit for bit.  The two device paths were written from the same rule, so each result is
also compared, bit for bit, with the CPU oracle's.
"""
import numpy as np
import pytest
import torch

import oracle

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def nm():
    from paper_2507_17301_b200 import nm as mod
    return mod


def _both(nm, w, n, m, t):
    ref = nm.nm_prune(w, n, m, t)
    v_ref, i_ref = nm.nm_weights_export(ref)
    values = torch.full((ref.c_out, ref.kk), float("nan"), device="cuda")
    indices = torch.full((ref.n_tiles, ref.kk), 0xFFFF, dtype=torch.int32, device="cuda").to(torch.uint16)
    nm.nm_prune_noalloc(w, n, m, t, values, indices)
    torch.cuda.synchronize()
    assert torch.equal(indices.view(torch.int16), i_ref.view(torch.int16))
    assert torch.equal(values.view(torch.int32), v_ref.view(torch.int32))
    v_cpu, i_cpu = oracle.prune(w.cpu().numpy(), n, m, t)
    assert np.array_equal(indices.cpu().numpy(), i_cpu)
    assert np.array_equal(values.cpu().numpy().view(np.uint32), v_cpu.view(np.uint32))


def test_two_calls_in_a_row_match_nm_prune(nm):
    g = torch.Generator().manual_seed(41)
    big = torch.randn((256, 3, 3, 128), generator=g).cuda()      # 8 tiles x 1152 columns
    small = torch.randn((40, 3, 3, 6), generator=g).cuda()       # tail tile, tail group, fewer cells
    _both(nm, big, 2, 4, 32)
    _both(nm, small, 3, 4, 16)
    _both(nm, big, 1, 8, 64)                                     # and back up again


def test_non_finite_weights_stay_inside_the_callers_buffers(nm):
    # a NaN score ranks as +infinity, no group keeps more than N columns: the words after the index
    # array (guard words of the same allocation) are untouched and the result equals the oracle's
    g = torch.Generator().manual_seed(43)
    w = torch.randn((24, 1, 1, 32), generator=g)
    w[:, 0, 0, 28:] = float("nan")                               # the last group of every tile, whole
    w[3, 0, 0, 5] = float("nan")
    n, m, t = 2, 4, 8
    v_cpu, i_cpu = oracle.prune(w.numpy(), n, m, t)
    n_idx = i_cpu.size
    guard = 64
    ibuf = torch.full((n_idx + guard,), 0x7ABC, dtype=torch.int32, device="cuda").to(torch.uint16)
    values = torch.zeros(v_cpu.shape, device="cuda")
    nm.nm_prune_noalloc(w.cuda(), n, m, t, values, ibuf[:n_idx].view(i_cpu.shape))
    torch.cuda.synchronize()
    out = ibuf.cpu().numpy()
    assert np.array_equal(out[:n_idx].reshape(i_cpu.shape), i_cpu)
    assert (out[n_idx:] == 0x7ABC).all()
    assert np.array_equal(values.cpu().numpy().view(np.uint32), v_cpu.view(np.uint32))


def test_binding_refuses_undersized_outputs(nm):
    w = torch.zeros((16, 1, 1, 16), device="cuda")
    with pytest.raises(TypeError):
        nm.nm_prune_noalloc(w, 2, 4, 8, torch.empty((16, 7), device="cuda"),
                            torch.empty((2, 8), dtype=torch.uint16, device="cuda"))
    with pytest.raises(TypeError):
        nm.nm_prune_noalloc(w, 2, 4, 8, torch.empty((16, 8), device="cuda"),
                            torch.empty((1, 8), dtype=torch.uint16, device="cuda"))


def test_refuses_more_cells_than_the_builtin_scratch(nm):
    w = torch.zeros((1024, 1, 1, 1024), device="cuda")           # T = 1: 1024 * 1024 cells
    values = torch.empty((1024, 512), device="cuda")
    indices = torch.empty((1024, 512), dtype=torch.uint16, device="cuda")
    assert 1024 * 1024 > nm.NM_NOALLOC_MAX_CELLS
    with pytest.raises(nm.NmError) as e:
        nm.nm_prune_noalloc(w, 2, 4, 1, values, indices)
    assert e.value.status == nm.NM_ERR_UNSUPPORTED
    assert "scratch" in str(e.value)
    # the regular entry point still takes it, and the library is still usable
    nm.nm_prune(w, 2, 4, 1)
    _both(nm, torch.ones((8, 1, 1, 8), device="cuda"), 2, 4, 4)
