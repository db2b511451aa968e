"""The library only enqueues work (no allocation, no synchronisation inside a call), so a call can be captured into a CUDA
graph, the side stream of the panel pipeline included, and replayed."""
import numpy as np
import pytest
import torch

from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host  # noqa: E402


def test_zgemm2m_replays_from_a_cuda_graph_bit_for_bit():
    m, n, k, nmod = 300, 2304, 256, 16                     # 2304 columns: two panels, so the side stream is part of the capture
    A, B = inputs.complex_inputs(m, n, k, seed=71)
    A2, B2 = inputs.complex_inputs(m, n, k, seed=72)
    with Workspace(b.workspace_bytes(b.OP_ZGEMM, m, n, k, nmod)):
        dA, dB = to_dev(A), to_dev(B)
        C_direct = empty_dev(m, n, torch.complex128)
        C_graph = empty_dev(m, n, torch.complex128, fill=-1.0)
        b.zgemm2m(dA, dB, C_direct, nmod)                   # also creates the library's stream and events before the capture
        b.device_status()
        want = to_host(C_direct)
        s = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=s):
            b.zgemm2m(dA, dB, C_graph, nmod, stream=torch.cuda.current_stream())
        g.replay()
        torch.cuda.synchronize()
        b.device_status()
        assert (to_host(C_graph) == want).all()
        # new operand values in the same buffers: the replay recomputes everything, scale exponents included
        dA.copy_(to_dev(A2))
        dB.copy_(to_dev(B2))
        g.replay()
        torch.cuda.synchronize()
        b.zgemm2m(dA, dB, C_direct, nmod)
        b.device_status()
        assert (to_host(C_graph) == to_host(C_direct)).all()
        assert not (to_host(C_graph) == want).all()
