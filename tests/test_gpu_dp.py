"""Batch-sharded (data-parallel) stages on one GPU: the batch is cut into shards, every stage runs for
all shards before the exchange that follows it (an in-process stand-in for the collective), and the
result is compared with the CPU oracle on the WHOLE batch -- stage by stage, as for the unsharded
entry point: |g|max bit-exact, sigma rel 1e-5, counts exact given the GPU's sigma, classes and clip
values given the counts, codes bit-exact given the clip values (Algorithm 1; Eq. 11, 14, 15, Eq. 1).
The sharded weight gradient: integer partials added exactly, then Eq. 7."""
import numpy as np
import pytest
import torch

from oracle import cpu as O
from paper_2102_04782_b200 import api, parallel, synth

from helpers import codes_from_nchw, codes_to_nchw, dev_input, geom, padding_is_zero, scalar, ws_bytes

pytestmark = pytest.mark.gpu
REL = 1e-5

CASES = [
    # (N, C, H, W), bf16, images per shard
    ((8, 64, 14, 14), True, [4, 4]),
    ((6, 40, 9, 11), False, [3, 2, 1]),
    ((5, 300, 5, 7), True, [2, 3]),          # more channels than a block has threads
    ((7, 24, 12, 10), False, [1, 1, 1, 4]),
    ((4, 16, 6, 6), True, [4]),              # a single shard
]


def make_shards(g, bf16, split):
    N, C, H, W = g.shape
    shards, first = [], 0
    for n in split:
        d = dev_input(g[first:first + n], bf16, api.NHWC)
        Cp = api.padded_channels(C)
        sh = parallel.GradShard(
            dY=d, N_local=n, first_image=first,
            vq=torch.full((n, H, W, Cp), 77, dtype=torch.int8, device="cuda"),
            gq=torch.full((n, H, W, Cp), 77, dtype=torch.int8, device="cuda"),
            s_state=torch.zeros(C, device="cuda"), cls=torch.zeros(C, dtype=torch.uint8, device="cuda"),
            gmax_layer=torch.zeros(1, device="cuda"), ws=ws_bytes(api.dp_grad_workspace_bytes(C)))
        parallel.alloc_stage_buffers(sh, C, torch)
        shards.append(sh)
        first += n
    return shards


def run_lockstep(shards, C, H, W, N, params, has_prev, seed):
    """parallel.quantize_grad_sharded with the exchanges acting on all shards at once."""
    X = parallel.LockstepCollective
    M = N * H * W
    for sh in shards:
        parallel.stage_pivot(api, sh, C)
    X.broadcast([sh.pivot for sh in shards], src=0)
    for sh in shards:
        parallel.stage_moments(api, sh, C, H, W)
    X.all_max([sh.absmax for sh in shards])
    X.all_sum([sh.sums for sh in shards])
    for sh in shards:
        parallel.stage_sigma_count(api, sh, C, H, W, M, params)
    X.all_sum([sh.cnt for sh in shards])
    for sh in shards:
        parallel.stage_solve_codes(api, sh, C, H, W, M, params, has_prev, seed)
    torch.cuda.synchronize()


@pytest.mark.parametrize("shape,bf16,split", CASES)
def test_sharded_gradient_quantization_equals_the_whole_batch(shape, bf16, split):
    N, C, H, W = shape
    M = N * H * W
    g, _, _ = synth.channel_mixed_grad(N, C, H, W, seed=401)
    g2, _, _ = synth.channel_mixed_grad(N, C, H, W, seed=402)
    if bf16:
        g, g2 = synth.round_to_bf16(g), synth.round_to_bf16(g2)
    s_prev = None
    for t, gt in enumerate((g, g2)):                     # the second iteration reads the first one's clip values (Eq. 14)
        shards = make_shards(gt, bf16, split)
        if s_prev is not None:
            for sh in shards:
                sh.s_state.copy_(torch.from_numpy(s_prev).cuda())
        run_lockstep(shards, C, H, W, N, None, t > 0, 31 + t)
        absmax, mean, sigma, gl = O.channel_stats(gt)
        first = 0
        for sh in shards:
            np.testing.assert_array_equal(sh.absmax.cpu().numpy(), absmax)
            assert float(sh.gmax_layer.item()) == gl
            sg = sh.sigma.cpu().numpy()
            np.testing.assert_allclose(sg, sigma, rtol=REL, atol=0)
            assert np.all(np.abs(sh.mean.cpu().numpy() - mean) <= REL * np.maximum(sigma, 1e-30) + 1e-7 * np.abs(mean))
            # every rank holds the same scalars
            assert torch.equal(sh.sigma, shards[0].sigma) and torch.equal(sh.cnt, shards[0].cnt)
            assert torch.equal(sh.s_state, shards[0].s_state) and torch.equal(sh.cls, shards[0].cls)
            cnt = O.density_count(gt, sg)
            np.testing.assert_array_equal(sh.cnt.cpu().numpy(), cnt.astype(np.int64))
            s_or, cls_or = O.classify_clip(cnt, absmax, M, s_prev=s_prev)
            s_gpu = sh.s_state.cpu().numpy()
            np.testing.assert_array_equal(sh.cls.cpu().numpy(), cls_or)
            np.testing.assert_allclose(s_gpu, s_or, rtol=REL, atol=0)
            n = sh.N_local
            vq_o = O.quantize(gt, s_gpu, stochastic=True, seed=31 + t, stream=0)[first:first + n]
            gq_o = O.quantize(gt, gl, stochastic=True, seed=31 + t, stream=1)[first:first + n]
            np.testing.assert_array_equal(codes_to_nchw(sh.vq, C), vq_o)
            np.testing.assert_array_equal(codes_to_nchw(sh.gq, C), gq_o)
            assert padding_is_zero(sh.vq, C) and padding_is_zero(sh.gq, C)
            first += n
        s_prev = shards[0].s_state.cpu().numpy()
    assert api.get_device_status() == api.OK


def test_sharded_codes_equal_the_unsharded_entry_point():
    """Same clip values in, same codes out as dai8_quantize_grad on the whole tensor."""
    N, C, H, W = 6, 32, 10, 12
    g = synth.round_to_bf16(synth.channel_mixed_grad(N, C, H, W, seed=403)[0])
    shards = make_shards(g, True, [2, 4])
    run_lockstep(shards, C, H, W, N, None, False, 9)
    d = dev_input(g, True, api.NHWC)
    Cp = api.padded_channels(C)
    vq, gq = (torch.empty((N, H, W, Cp), dtype=torch.int8, device="cuda") for _ in range(2))
    s_state, gmax, cls = torch.zeros(C, device="cuda"), torch.zeros(1, device="cuda"), torch.zeros(C, dtype=torch.uint8, device="cuda")
    api.quantize_grad(d, api.NHWC, N, C, H, W, None, s_state, False, gmax, None, cls, vq, gq, 9,
                      ws_bytes(api.quantize_grad_workspace_bytes(C)))
    torch.cuda.synchronize()
    if torch.equal(s_state, shards[0].s_state):          # identical clip values (sigma may differ in the last place)
        assert torch.equal(torch.cat([sh.vq for sh in shards]), vq)
    assert torch.equal(torch.cat([sh.gq for sh in shards]), gq)
    assert torch.equal(gmax, shards[0].gmax_layer) and torch.equal(cls, shards[0].cls)


def test_sharded_weight_gradient_and_activation_scale():
    rng = np.random.default_rng(404)
    N, Cin, Cout, H, W, R, S, st, pad = 6, 24, 40, 13, 11, 3, 3, 1, 1
    split = [1, 3, 2]
    x = (synth.activations(N, Cin, H, W, seed=405) - np.float32(0.2)).astype(np.float32)
    P, Q = O.out_hw(H, W, R, S, st, pad)
    vq_all = rng.integers(-127, 128, size=(N, Cout, P, Q), dtype=np.int64).astype(np.int8)
    s_c = (10.0 ** rng.uniform(-6, -3, Cout)).astype(np.float32)
    X = parallel.LockstepCollective
    # activation scale of the whole batch, then codes per shard
    sXs, qXs, first = [], [], 0
    for n in split:
        d = dev_input(x[first:first + n], False, api.NHWC)
        sX = torch.zeros(1, device="cuda")
        api.absmax(d, sX)
        sXs.append(sX); qXs.append(d)
        first += n
    X.all_max(sXs)
    assert float(sXs[0].item()) == float(np.abs(x).max())
    Cp = api.padded_channels(Cin)
    codes, first = [], 0
    for n, d, sX in zip(split, qXs, sXs):
        q = torch.empty((n, H, W, Cp), dtype=torch.int8, device="cuda")
        api.quantize_tensor(d, api.NHWC, n, Cin, H, W, api.SCALE_GIVEN, sX, api.ROUND_NEAREST_EVEN, 0, q)
        codes.append(q)
        first += n
    qx_o = O.quantize(x, float(sXs[0].item()))
    np.testing.assert_array_equal(np.concatenate([codes_to_nchw(q, Cin) for q in codes]), qx_o)
    # integer partials of dW per shard, exact sum, Eq. 7
    accs, first = [], 0
    s_dev = torch.from_numpy(s_c).cuda()
    for n, q in zip(split, codes):
        gm = geom(n, Cin, Cout, H, W, R, S, st, pad)
        acc = torch.empty((Cout, Cin, R, S), dtype=torch.int32, device="cuda")
        api.conv_bwd_filter(q, codes_from_nchw(vq_all[first:first + n]), sXs[0], s_dev, gm, acc,
                            ws_bytes(max(16, api.conv_workspace_bytes(api.OP_BWD_FILTER, gm))))
        accs.append(acc)
        first += n
    X.all_sum(accs)
    acc_o, overflow = O.conv_bwd_filter_acc(qx_o, vq_all, (R, S), st, pad)
    assert overflow == 0
    np.testing.assert_array_equal(accs[0].cpu().numpy(), acc_o)
    dW = torch.empty((Cout, Cin, R, S), dtype=torch.float32, device="cuda")
    api.dequant_filter(accs[0], sXs[0], s_dev, Cout, Cin * R * S, dW)
    want = O.dequant_acc(acc_o, float(sXs[0].item()), s_c)
    got = dW.cpu().numpy()
    for co in range(Cout):
        assert np.abs(got[co] - want[co]).max() <= REL * np.abs(want[co]).max() + 1e-45
    assert api.get_device_status() == api.OK


def test_rejections():
    C = 16
    t = torch.zeros(4 * 4 * C, device="cuda")
    f = torch.zeros(C, device="cuda")
    with pytest.raises(api.Dai8Error) as e:
        api.dp_grad_moments(t, api.NCHW, 1, C, 4, 4, f, f, torch.zeros(2 * C, dtype=torch.float64, device="cuda"),
                            ws_bytes(api.dp_grad_workspace_bytes(C)))
    assert e.value.code == api.ERR_UNSUPPORTED
    with pytest.raises(api.Dai8Error) as e:
        api.dp_grad_moments(t, api.NHWC, 1, C, 4, 4, f, f, torch.zeros(2 * C, dtype=torch.float64, device="cuda"), ws_bytes(64))
    assert e.value.code == api.ERR_WORKSPACE
