"""fvattn_sparse_attn_noalloc: the attention call for hosts that cannot allocate device memory
(all of it already sits in their own arena, or cudaMalloc's device-wide synchronisation is not
acceptable where they call from).  It keeps its scratch in a fixed array inside the library, takes
no workspace, and must give exactly what fvattn_sparse_attn gives.  The array is shared and keeps
the previous call's contents, so the check runs twice in a row, the second time on a different
mask.  Collected last (file name), so a failure here cannot hide any other test's result; it
builds its own inputs, so it also passes when run alone in a fresh process."""
import ctypes

import pytest
import torch

from paper_2607_16190_b200 import binding as fv
from paper_2607_16190_b200 import synth

pytestmark = pytest.mark.gpu


def _inputs(name):
    cfg = synth.CONFIGS[name]
    q, k, v, _ = synth.make_qkv(cfg, "cuda")
    g = fv.Grid(*cfg.grid, *cfg.tile)
    q_r, k_r, v_r = (fv.reorder(t, g) for t in (q, k, v))
    return cfg, g, q_r, k_r, v_r


@pytest.mark.parametrize("name", ["small", "tiny"])
def test_noalloc_matches_workspace_entry_point_twice_in_a_row(name):
    cfg, g, q_r, k_r, v_r = _inputs(name)
    ws = fv.make_workspace(g, 1, cfg.H, cfg.d)
    out = torch.empty_like(q_r)
    status = torch.full((2,), 77, dtype=torch.uint32, device="cuda")
    for p, k_floor in ((cfg.p, cfg.k_floor), (0.5, 1)):           # two calls in a row, different masks
        routing = fv.route(q_r, k_r, g, p, k_floor, cfg.sm_scale, ws)
        want = fv.sparse_attn(q_r, k_r, v_r, routing.idx, routing.counts, g, cfg.sm_scale, ws)
        assert fv.device_status(ws) == fv.OK
        out.fill_(float("nan"))
        fv.sparse_attn_noalloc(q_r, k_r, v_r, routing.idx, routing.counts, g, cfg.sm_scale, out, status)
        torch.cuda.synchronize()
        assert status.cpu().view(torch.int32).tolist() == [0, 0]
        # same kernels, same inputs, each output row written by one CTA: bit-identical
        assert torch.equal(out, want)


def test_noalloc_rejects_shapes_beyond_its_fixed_scratch_and_bad_arguments():
    L = fv.lib()
    fake = ctypes.c_void_p(0x100000)      # never dereferenced: validation fails before any launch
    null = ctypes.c_void_p(0)
    big = fv.Grid(64, 64, 128, 1, 8, 16).c()                       # nb = 4096 blocks, 128 heads: > 1 MiB of scratch
    st = L.fvattn_sparse_attn_noalloc(fake, fake, fake, fake, fake, 1, 128, 128, ctypes.byref(big),
                                      ctypes.c_float(0.1), fake, null, null)
    assert st == fv.ERR_WORKSPACE_TOO_SMALL
    small = fv.Grid(8, 16, 16, 2, 8, 8).c()
    st = L.fvattn_sparse_attn_noalloc(null, fake, fake, fake, fake, 1, 12, 128, ctypes.byref(small),
                                      ctypes.c_float(0.1), fake, null, null)
    assert st == fv.ERR_INVALID_ARG
