"""dai8_quantize_grad_noalloc against dai8_quantize_grad.

Some users of the library cannot allocate device memory at the point where they quantize the
gradient (they are handed only their input and output tensors, or all device memory was given out at
start-up, or an allocation would stall the device in a latency-critical loop).  For them the library
has a variant whose scratch memory is a fixed array inside the library image.  This test calls that
variant through the C ABI twice in a row (the second call on a different tensor, with the first
call's clip state, so anything stale left in the shared scratch would show) and requires every
output to equal the one of the ordinary entry point: integers and codes bit for bit, clip values and
statistics within the relative 1e-5 the other GPU tests use.

The file name sorts last on purpose: if this test fails under `-x`, every other test has already run.
"""
import numpy as np
import pytest
import torch

from paper_2102_04782_b200 import api, synth

from helpers import GradQuant, dev_input

pytestmark = pytest.mark.gpu

REL = 1e-5


class NoAllocBuffers(GradQuant):
    def run_noalloc(self, dY, layout, seed, has_prev):
        api.quantize_grad_noalloc(dY, layout, self.N, self.C, self.H, self.W, None, self.s_state,
                                  has_prev, self.gmax, self.stats, self.cls, self.vq, self.gq, seed)
        torch.cuda.synchronize()


def outputs(b):
    return (b.vq.cpu().numpy().copy(), b.gq.cpu().numpy().copy(), b.cls.cpu().numpy().copy(),
            b.gmax.cpu().numpy().copy(), b.s_state.cpu().numpy().copy(), b.stats.cpu().numpy().copy())


@pytest.mark.parametrize("layout", [api.NHWC, api.NCHW])
@pytest.mark.parametrize("shape,bf16", [((8, 64, 14, 14), False), ((4, 256, 28, 28), True),
                                        ((3, 20, 5, 7), True)])
def test_noalloc_matches_workspace_entry_point(shape, bf16, layout):
    N, C, H, W = shape
    tensors = []
    for seed in (21, 22):
        g, _, _ = synth.channel_mixed_grad(N, C, H, W, seed=seed)
        if bf16:
            g = synth.round_to_bf16(g)
        tensors.append(dev_input(g, bf16, layout))
    ref, got = GradQuant(N, C, H, W), NoAllocBuffers(N, C, H, W)
    for t, d in enumerate(tensors):               # two calls in a row on the shared scratch
        ref.run(d, layout, 100 + t, has_prev=t > 0)
        got.run_noalloc(d, layout, 100 + t, has_prev=t > 0)
        r, o = outputs(ref), outputs(got)
        for a, b in zip(r[:4], o[:4]):            # codes, classes, layer |g|max: exact
            np.testing.assert_array_equal(a, b)
        np.testing.assert_allclose(o[4], r[4], rtol=REL, atol=0)     # clip values
        np.testing.assert_allclose(o[5], r[5], rtol=REL, atol=1e-12)  # |g|max, mean, sigma, P
    assert api.get_device_status() == api.OK


def test_noalloc_rejects_more_channels_than_the_scratch_holds():
    C = api.NOALLOC_MAX_CHANNELS + 16
    b = NoAllocBuffers(1, C, 2, 2)
    before = api.launch_count()
    with pytest.raises(api.Dai8Error) as e:
        b.run_noalloc(torch.zeros((1, 2, 2, C), dtype=torch.float32, device="cuda"), api.NHWC, 0, False)
    assert e.value.code == api.ERR_WORKSPACE
    assert api.launch_count() == before           # nothing was enqueued
