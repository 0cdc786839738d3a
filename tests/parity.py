"""Shared helpers for the GPU parity tests: run one layer through the C-ABI binding and through
the CPU oracle on the same seeded inputs and compare (helpers only; no method arithmetic)."""
import numpy as np
import torch

import oracle
from paper_2507_17301_b200 import inputs

REL_FRO_TOL = 2e-3      # relative Frobenius error allowed under TF32
MAX_ABS_TOL = 1e-2      # max-abs error allowed, as a fraction of max|ref|


def tensors_for(s: inputs.ConvShape, integer: bool = False, layer: int = 0):
    if integer:
        return inputs.make_int_case(s, layer)
    return inputs.make_weights(s, layer), inputs.make_activations(s, layer), inputs.make_bias(s, layer)


def oracle_layer(s: inputs.ConvShape, w, x, b, use_bias=True):
    values, indices = oracle.prune(w.numpy(), s.n_keep, s.m_group, s.tile_t)
    y = oracle.conv2d(values, indices, s.kh, s.kw, s.c_in, s.tile_t, x.numpy(), (s.stride, s.stride),
                      (s.pad, s.pad), (s.dil, s.dil), b.numpy() if use_bias else None, s.relu)
    return values, indices, y


def gpu_layer(nm, s: inputs.ConvShape, w, x, b, use_bias=True, plan=None):
    wd = w.cuda()
    hnd = nm.nm_prune(wd, s.n_keep, s.m_group, s.tile_t)
    values, indices = nm.nm_weights_export(hnd)
    y = nm.nm_conv2d(hnd, x.cuda(), s.kh, s.kw, s.stride, s.pad, s.dil, b.cuda() if use_bias else None, s.relu,
                     plan=plan)
    nm.nm_weights_check(hnd)
    torch.cuda.synchronize()
    return hnd, values.cpu().numpy(), indices.cpu().numpy(), y.cpu().numpy()


def assert_prune_bit_exact(values_gpu, indices_gpu, values_ref, indices_ref):
    assert indices_gpu.shape == indices_ref.shape and values_gpu.shape == values_ref.shape
    assert np.array_equal(indices_gpu, indices_ref), "retained-column indices differ from the oracle"
    assert np.array_equal(values_gpu.view(np.uint32), values_ref.view(np.uint32)), "compacted values differ"


def errors(y_gpu, y_ref):
    d = y_gpu.astype(np.float64) - y_ref.astype(np.float64)
    ref_n = float(np.sqrt((y_ref.astype(np.float64) ** 2).sum()))
    rel_fro = float(np.sqrt((d ** 2).sum())) / max(ref_n, 1e-30)
    max_abs = float(np.abs(d).max()) if d.size else 0.0
    ref_max = float(np.abs(y_ref).max()) if d.size else 0.0
    return rel_fro, max_abs, ref_max


def assert_conv_close(y_gpu, y_ref):
    assert y_gpu.shape == y_ref.shape
    assert np.isfinite(y_gpu).all()
    rel_fro, max_abs, ref_max = errors(y_gpu, y_ref)
    assert rel_fro <= REL_FRO_TOL, f"relative Frobenius error {rel_fro:.3e} above {REL_FRO_TOL}"
    assert max_abs <= MAX_ABS_TOL * ref_max, f"max-abs error {max_abs:.3e} above {MAX_ABS_TOL} * {ref_max:.3e}"
