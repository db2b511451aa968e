"""The library only enqueues work (no allocation, no synchronisation inside a call), so a call can be captured into a CUDA
graph, the side stream of the panel pipeline included, and replayed."""
import numpy as np
import pytest
import torch

from paper_2609_05419_b200 import binding as b
from paper_2609_05419_b200 import inputs

pytestmark = pytest.mark.gpu

from gpu_util import Workspace, empty_dev, to_dev, to_host  # noqa: E402


@pytest.mark.parametrize("overlap", [False, True], ids=["in-order", "overlap"])
def test_zgemm2m_replays_from_a_cuda_graph_bit_for_bit(overlap):
    m, n, k, nmod = 300, 2304, 256, 16                     # 2304 columns: two panels; with the overlap on, the library's stream is part of the capture
    A, B = inputs.complex_inputs(m, n, k, seed=71)
    A2, B2 = inputs.complex_inputs(m, n, k, seed=72)
    b.debug_set_overlap(overlap)
    try:
        _replay_case(m, n, k, nmod, A, B, A2, B2)
    finally:
        b.debug_set_overlap(False)


def _replay_case(m, n, k, nmod, A, B, A2, B2):
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


def test_host_form_and_eisenstein_variant_replay_from_a_cuda_graph():
    m, n, k, nmod = 260, 700, 200, 16                      # 700 columns: two panels of the host form, three streams in the capture
    A, B = inputs.complex_inputs(m, n, k, seed=73)
    A2, B2 = inputs.complex_inputs(m, n, k, seed=74)
    pin = lambda x: torch.from_numpy(np.ascontiguousarray(x.T)).pin_memory().t()
    hA, hB = pin(A), pin(B)
    hC = torch.empty((n, m), dtype=torch.complex128).pin_memory().t()
    with Workspace(b.workspace_bytes(b.OP_ZGEMM_HOST, m, n, k, nmod)):
        dA, dB = to_dev(A), to_dev(B)
        C_dev = empty_dev(m, n, torch.complex128)
        C_eis = empty_dev(m, n, torch.complex128)
        b.zgemm2m_host(hA, hB, hC, nmod)                    # first calls outside the capture: they create streams and events
        b.zgemm2m_eisenstein(dA, dB, C_eis, nmod)
        torch.cuda.synchronize()
        b.device_status()
        want_host, want_eis = hC.numpy().copy(), to_host(C_eis)
        hC.fill_(0)
        C_eis.fill_(0)
        s = torch.cuda.Stream()
        g = torch.cuda.CUDAGraph()
        s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.graph(g, stream=s):
            b.zgemm2m_host(hA, hB, hC, nmod, stream=torch.cuda.current_stream())
            b.zgemm2m_eisenstein(dA, dB, C_eis, nmod, stream=torch.cuda.current_stream())
        g.replay()
        torch.cuda.synchronize()
        b.device_status()
        assert (hC.numpy() == want_host).all() and (to_host(C_eis) == want_eis).all()
        hA.copy_(torch.from_numpy(np.ascontiguousarray(A2)))       # new values in the same host buffers
        hB.copy_(torch.from_numpy(np.ascontiguousarray(B2)))
        g.replay()
        torch.cuda.synchronize()
        b.zgemm2m(to_dev(A2), to_dev(B2), C_dev, nmod)
        b.device_status()
        assert (hC.numpy() == to_host(C_dev)).all() and not (hC.numpy() == want_host).all()
