"""The entry points enqueue kernels only (no allocation, no synchronisation), so a forward + backward step
can be captured once into a CUDA graph and replayed."""
import pytest
import torch

from paper_2609_19242_b200 import binding, synth
from paper_2609_19242_b200.synth import Workload

import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("fused", [False, True], ids=["two_pass", "fused"])
def test_forward_backward_replay_from_a_cuda_graph(fused):
    w = Workload("graph", 1, 4, 2, 128, 512, 32)
    g = pu.to_cuda(synth.make_inputs(w, "cpu"))
    M = w.block_size
    args = [g[n] for n in pu.NAMES6]
    # eager reference (also performs the library's one-time per-device setup outside the capture)
    ref_o = binding.bdlm_attn_fwd(*args, M)
    ref_g = binding.bdlm_attn_bwd(*args, ref_o[0], ref_o[1], ref_o[2], ref_o[3], g["do_clean"], g["do_noisy"], M,
                                  single_pass=fused)
    torch.cuda.synchronize()
    out = tuple(torch.zeros_like(t) for t in ref_o)
    grads = tuple(torch.zeros_like(t) for t in ref_g)
    p = binding.make_params(w.batch, w.L, M, w.H, w.H_kv, w.d, bwd_single_pass=fused)
    ws = torch.empty(binding.bdlm_workspace_bytes(p, binding.BDLM_WS_BWD), dtype=torch.uint8, device="cuda")
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.bdlm_attn_fwd(*args, M, out=out)
        binding.bdlm_attn_bwd(*args, out[0], out[1], out[2], out[3], g["do_clean"], g["do_noisy"], M,
                              out=grads, workspace=ws, single_pass=fused)
    for t in out + grads:
        t.zero_()
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert binding.bdlm_get_device_status() == 0
    for i, (a, b) in enumerate(zip(out + grads, ref_o + ref_g)):
        if fused and i in (4, 7):   # dQ of the fused backward: fp32 summation order of the key tiles' reductions
            assert pu.rel_l2(synth.to_f64(a), synth.to_f64(b)) <= 1e-3
        else:
            assert torch.equal(a, b)
    # new inputs in the same buffers, same graph
    g["q_clean"].copy_(g["q_clean"].flip(1))
    ref_o2 = binding.bdlm_attn_fwd(*args, M)
    graph.replay()
    torch.cuda.synchronize()
    assert torch.equal(out[0], ref_o2[0]) and torch.equal(out[1], ref_o2[1])
