"""Every entry point only enqueues work on the caller's stream (no allocation, no synchronisation, no
host read of device results), so a layer step can be captured in a CUDA graph and replayed.  The replay
must reproduce the eager results bit for bit, for the small-tensor kernels and for the cooperative /
tensor-core ones."""
import pytest
import torch

from paper_2102_04782_b200 import api, synth

pytestmark = pytest.mark.gpu

LAYERS = [
    (synth.config1_layer(), 8),
    (synth.ConvLayer("conv3x3_64_32x40", 64, 64, 32, 40, 3, 3, 1, 1), 4),
    (synth.ConvLayer("conv1x1_96_24_28", 96, 24, 28, 28, 1, 1, 1, 0), 6),
]


@pytest.mark.parametrize("L,N", LAYERS, ids=lambda v: getattr(v, "name", str(v)))
def test_a_captured_layer_step_replays_bit_exactly(L, N):
    dev = "cuda"
    x, w, g = synth.device_layer_inputs(L, N, 301, torch.device(dev))
    geom = api.ConvGeom(N, L.Cin, L.Cout, L.H, L.W, L.R, L.S, L.stride, L.stride, L.pad, L.pad)
    Cp, Cop = api.padded_channels(L.Cin), api.padded_channels(L.Cout)
    i8, f32 = dict(dtype=torch.int8, device=dev), dict(dtype=torch.float32, device=dev)
    qX, qW = torch.empty((N, L.H, L.W, Cp), **i8), torch.empty((L.Cout, L.R, L.S, Cp), **i8)
    vq, gq = torch.empty((N, L.P, L.Q, Cop), **i8), torch.empty((N, L.P, L.Q, Cop), **i8)
    sX, sW, gmax = torch.zeros(1, **f32), torch.zeros(1, **f32), torch.zeros(1, **f32)
    s_state = torch.zeros(L.Cout, **f32)
    Y = torch.empty((N, L.P, L.Q, L.Cout), **f32)
    dX = torch.empty((N, L.H, L.W, L.Cin), **f32)
    dW = torch.empty((L.Cout, L.Cin, L.R, L.S), **f32)

    def ws(n):
        return torch.empty(max(n, 16), dtype=torch.uint8, device=dev)

    ws_q, ws_g = ws(api.quantize_tensor_workspace_bytes()), ws(api.quantize_grad_workspace_bytes(L.Cout))
    ws_f, ws_d, ws_w = (ws(api.conv_workspace_bytes(op, geom)) for op in (api.OP_FWD, api.OP_BWD_DATA, api.OP_BWD_FILTER))

    def step():
        api.quantize_tensor(x, api.NHWC, N, L.Cin, L.H, L.W, api.SCALE_ABSMAX, sX, api.ROUND_NEAREST_EVEN, 0, qX, ws_q)
        api.quantize_tensor(w, api.NCHW, L.Cout, L.Cin, L.R, L.S, api.SCALE_ABSMAX, sW, api.ROUND_NEAREST_EVEN, 0, qW, ws_q)
        api.conv_fwd(qX, qW, sX, sW, geom, Y, api.NHWC, ws_f)
        api.quantize_grad(g, api.NHWC, N, L.Cout, L.P, L.Q, None, s_state, True, gmax, None, None, vq, gq, 9, ws_g)
        api.conv_bwd_filter(qX, vq, sX, s_state, geom, dW, ws_w)
        api.conv_bwd_data(gq, qW, gmax, sW, geom, dX, api.NHWC, ws_d)

    outs = (qX, qW, vq, gq, sX, sW, gmax, s_state, Y, dX, dW)
    s0 = torch.full((L.Cout,), 1e-4, **f32)      # the clip values of the previous iteration (Eq. 14 reads them)
    s_state.copy_(s0)
    step()                                       # eager; also first-use initialisation, outside the capture
    torch.cuda.synchronize()
    want = [t.clone() for t in outs]
    graph = torch.cuda.CUDAGraph()
    s_state.copy_(s0)
    with torch.cuda.graph(graph):
        step()
    for replay in range(2):
        for t in outs:
            t.zero_()
        s_state.copy_(s0)
        graph.replay()
        torch.cuda.synchronize()
        for a, b in zip(outs, want):
            assert torch.equal(a, b), f"replay {replay}"
    assert api.get_device_status() == api.OK
