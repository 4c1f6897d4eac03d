"""The tile scheduler enumerates exactly the 128x128 tiles that contain a visible (query, key) pair:
the kernels' own step counters (bdlm_set_trace_buffer) are compared with counts taken from the
oracle's explicit mask."""
import numpy as np
import pytest
import torch

from oracle import bdlm_oracle as orc
from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import Workload

import parity_util as pu

pytestmark = pytest.mark.gpu


def _tiles_with_a_visible_pair(L, M, T=128):
    vis = orc.visibility_2L(L, M)
    n = L // T
    t = vis.reshape(2, n, T, 2, n, T).any(axis=(2, 5))     # [q stream, q tile, k stream, k tile]
    return int(t.sum())


@pytest.mark.parametrize("L,M", [(512, 32), (640, 128), (1024, 256), (512, 16), (384, 64)])
def test_step_counts_equal_unmasked_tile_counts(L, M):
    w = Workload("sched", 2, 4, 2, 128, L, M)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    tr = torch.zeros(binding.TRACE_SLOTS, dtype=torch.int64, device="cuda")
    binding.bdlm_set_trace_buffer(tr)
    try:
        out = pu.gpu_fwd(g, M, impl=binding.IMPL_TCGEN05)
        pu.gpu_bwd(g, out, M, impl=binding.IMPL_TCGEN05)
        torch.cuda.synchronize()
    finally:
        binding.bdlm_set_trace_buffer(None)
    t = tr.cpu().tolist()
    tiles = _tiles_with_a_visible_pair(L, M)
    assert t[0] == tiles * w.batch * w.H // 2      # forward: one CTA walks the tiles of two heads at once
    assert t[16] == tiles * w.batch * w.H          # dK/dV pass: every (key tile, query tile, head)
    assert t[32] == tiles * w.batch * w.H          # dQ pass
    assert t[6] > 0 and t[16 + 6] > 0 and t[32 + 6] > 0   # cycle counters were written
    assert binding.bdlm_get_device_status() == 0
