"""The N > 1 path of bench.py is "replicas only": no data-path collective, just the max over ranks
of the step time and the summed throughput.  Exercised here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")      # rank 1 is the slow replica
    dist.barrier()
    out[rank] = (ms, bench.aggregate_value(2e12, ms, world))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_two_gloo_ranks():
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(2, 29731, out), nprocs=2, join=True)
        assert out[0] == out[1]
        ms, value = out[0]
        assert ms == 15.0                                   # the slowest replica sets the time
        assert abs(value - 2 * 2e12 / 15e-3 / 1e12) < 1e-9   # both replicas' work counts


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5) == 3.5
    assert bench.aggregate_value(1e12, 1.0, 1) == 1000.0


def test_reference_arm_prints_on_rank_zero_only():
    """`--impl reference` under a 2-rank launch: rank 1 exits 0 without output."""
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


# ---- the batch-sharded step over a real process group (gloo, two ranks, CPU) -------------------------
class _OracleStages:
    """Stand-in for the binding module in parallel.py: the same stage calls, computed by the CPU oracle
    on CPU tensors, so that the orchestration and its exchanges run over gloo without a GPU."""
    NHWC = 1

    def __init__(self):
        sys.path.insert(0, ROOT)
        from oracle import cpu as O
        import numpy as np
        self.O, self.np = O, np

    def _nchw(self, dY, N, C, H, W):
        return self.np.ascontiguousarray(dY.numpy().reshape(N, H, W, C).transpose(0, 3, 1, 2))

    def dp_grad_pivot(self, dY, layout, C, pivot):
        pivot.copy_(dY.reshape(-1, C)[0])

    def dp_grad_moments(self, dY, layout, N, C, H, W, pivot, absmax, sums, ws):
        np = self.np
        g = self._nchw(dY, N, C, H, W).astype(np.float64)
        d = g - pivot.numpy().astype(np.float64)[None, :, None, None]
        absmax.copy_(torch.from_numpy(np.abs(g).max(axis=(0, 2, 3)).astype(np.float32)))
        sums.copy_(torch.from_numpy(np.concatenate([d.sum(axis=(0, 2, 3)), (d * d).sum(axis=(0, 2, 3))])))

    def dp_grad_sigma(self, absmax, sums, pivot, C, M, params, mean, sigma, gmax_layer):
        np = self.np
        s1, s2 = sums.numpy()[:C], sums.numpy()[C:]
        md = s1 / M
        mean.copy_(torch.from_numpy((pivot.numpy().astype(np.float64) + md).astype(np.float32)))
        sigma.copy_(torch.from_numpy(np.sqrt(np.maximum(s2 - s1 * md, 0.0) / M).astype(np.float32)))
        gmax_layer.copy_(absmax.max().reshape(1))

    def dp_grad_count(self, dY, layout, N, C, H, W, sigma, cnt, ws):
        cnt.copy_(torch.from_numpy(self.O.density_count(self._nchw(dY, N, C, H, W), sigma.numpy()).astype(self.np.int64)))

    def dp_grad_solve(self, cnt, absmax, C, M, params, s_state, has_prev, cls):
        s, c = self.O.classify_clip(cnt.numpy(), absmax.numpy(), M, s_prev=s_state.numpy().copy() if has_prev else None)
        s_state.copy_(torch.from_numpy(s)); cls.copy_(torch.from_numpy(c))

    def dp_grad_codes(self, dY, layout, N, C, H, W, first_image, s, gmax_layer, seed, vq, gq):
        g = self._nchw(dY, N, C, H, W)
        a = self.O.quantize(g, s.numpy(), True, seed, 0, first_image=first_image)
        b = self.O.quantize(g, float(gmax_layer.item()), True, seed, 1, first_image=first_image)
        vq.copy_(torch.from_numpy(a.transpose(0, 2, 3, 1).copy())); gq.copy_(torch.from_numpy(b.transpose(0, 2, 3, 1).copy()))


def _dp_worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2102_04782_b200 import parallel, synth
    dist.init_process_group("gloo", rank=rank, world_size=world)
    N, C, H, W = 6, 12, 7, 5
    split = [4, 2]
    g = synth.channel_mixed_grad(N, C, H, W, seed=77)[0]
    first = sum(split[:rank]); n = split[rank]
    dY = torch.from_numpy(np.ascontiguousarray(g[first:first + n].transpose(0, 2, 3, 1)))
    sh = parallel.GradShard(dY=dY, N_local=n, first_image=first, vq=torch.zeros((n, H, W, C), dtype=torch.int8),
                            gq=torch.zeros((n, H, W, C), dtype=torch.int8), s_state=torch.full((C,), 2e-4),
                            cls=torch.zeros(C, dtype=torch.uint8), gmax_layer=torch.zeros(1), ws=None)
    parallel.alloc_stage_buffers(sh, C, torch)
    parallel.quantize_grad_sharded(_OracleStages(), parallel.Collective(dist), sh, C, H, W, N, None, True, 5)
    # the weight-gradient exchange: an exact integer sum
    acc = torch.full((3, 4), rank + 1, dtype=torch.int32)
    parallel.Collective(dist).all_sum(acc)
    out[rank] = (sh.s_state.numpy().copy(), sh.cls.numpy().copy(), float(sh.gmax_layer.item()), sh.sigma.numpy().copy(),
                 sh.vq.numpy().copy(), sh.gq.numpy().copy(), acc.numpy().copy())
    dist.destroy_process_group()


def test_sharded_gradient_quantization_two_gloo_ranks():
    """Two ranks with 4 and 2 images: after the exchanges both hold the whole batch's statistics, classes
    and clip values, and their codes are the whole-batch oracle's codes of their images."""
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import cpu as O
    from paper_2102_04782_b200 import synth
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_dp_worker, args=(2, 29741, out), nprocs=2, join=True)
        r0, r1 = out[0], out[1]
    N, C, H, W = 6, 12, 7, 5
    g = synth.channel_mixed_grad(N, C, H, W, seed=77)[0]
    absmax, mean, sigma, gl = O.channel_stats(g)
    for a, b in zip(r0[:4], r1[:4]):
        assert np.array_equal(a, b)                          # identical scalars on both ranks
    assert r0[2] == gl
    np.testing.assert_allclose(r0[3], sigma, rtol=1e-6)
    cnt = O.density_count(g, r0[3])
    s, cls = O.classify_clip(cnt, absmax, N * H * W, s_prev=np.full(C, 2e-4, np.float32))
    np.testing.assert_array_equal(r0[1], cls)
    np.testing.assert_allclose(r0[0], s, rtol=1e-6)
    vq = O.quantize(g, r0[0], True, 5, 0).transpose(0, 2, 3, 1)
    gq = O.quantize(g, gl, True, 5, 1).transpose(0, 2, 3, 1)
    np.testing.assert_array_equal(np.concatenate([r0[4], r1[4]]), vq)
    np.testing.assert_array_equal(np.concatenate([r0[5], r1[5]]), gq)
    assert np.array_equal(r0[6], np.full((3, 4), 3, np.int32)) and np.array_equal(r1[6], r0[6])
