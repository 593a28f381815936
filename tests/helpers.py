"""Layout conversions and device plumbing shared by the GPU parity tests (no method arithmetic)."""
from __future__ import annotations

import numpy as np
import torch

from paper_2102_04782_b200 import api


def dev_input(x_nchw: np.ndarray, bf16: bool, layout: int) -> torch.Tensor:
    """fp32 NCHW numpy -> CUDA tensor in the requested dtype / layout (values must already be
    bf16-representable when bf16 is requested, so the cast is exact)."""
    t = torch.from_numpy(np.ascontiguousarray(x_nchw))
    if layout == api.NHWC:
        t = t.permute(0, 2, 3, 1).contiguous()
    t = t.cuda()
    if bf16:
        t = t.to(torch.bfloat16)
    return t.contiguous()


def codes_to_nchw(q_dev: torch.Tensor, C: int) -> np.ndarray:
    """int8 [N][H][W][Cp] device codes -> NCHW numpy (padding channels dropped)."""
    return np.ascontiguousarray(q_dev.cpu().numpy()[..., :C].transpose(0, 3, 1, 2))


def padding_is_zero(q_dev: torch.Tensor, C: int) -> bool:
    return bool((q_dev[..., C:] == 0).all().item())


def codes_from_nchw(q_nchw: np.ndarray) -> torch.Tensor:
    """NCHW int8 numpy -> device [N][H][W][Cp] with zero padding channels."""
    N, C, H, W = q_nchw.shape
    Cp = (C + 15) // 16 * 16
    out = np.zeros((N, H, W, Cp), np.int8)
    out[..., :C] = q_nchw.transpose(0, 2, 3, 1)
    return torch.from_numpy(out).cuda()


def out_to_nchw(t: torch.Tensor, layout: int) -> np.ndarray:
    a = t.float().cpu().numpy() if t.dtype == torch.bfloat16 else t.cpu().numpy()
    if layout == api.NHWC:
        a = a.transpose(0, 3, 1, 2)
    return np.ascontiguousarray(a)


def geom(N, Cin, Cout, H, W, R, S, stride, pad) -> api.ConvGeom:
    sh, sw = (stride, stride) if np.isscalar(stride) else stride
    ph, pw = (pad, pad) if np.isscalar(pad) else pad
    return api.ConvGeom(N, Cin, Cout, H, W, R, S, sh, sw, ph, pw)


def scalar(v: float) -> torch.Tensor:
    return torch.tensor([v], dtype=torch.float32, device="cuda")


def ws_bytes(n: int) -> torch.Tensor:
    return torch.empty(max(n, 16), dtype=torch.uint8, device="cuda")


class GradQuant:
    """Device buffers for one dai8_quantize_grad call."""

    def __init__(self, N, C, H, W):
        self.N, self.C, self.H, self.W = N, C, H, W
        Cp = api.padded_channels(C)
        d = "cuda"
        self.s_state = torch.zeros(C, dtype=torch.float32, device=d)
        self.gmax = torch.zeros(1, dtype=torch.float32, device=d)
        self.stats = torch.zeros(C, 4, dtype=torch.float32, device=d)
        self.cls = torch.zeros(C, dtype=torch.uint8, device=d)
        self.vq = torch.full((N, H, W, Cp), 77, dtype=torch.int8, device=d)
        self.gq = torch.full((N, H, W, Cp), 77, dtype=torch.int8, device=d)
        self.ws = ws_bytes(api.quantize_grad_workspace_bytes(C))

    def run(self, dY, layout, seed, has_prev, params=None, sigma_override=None, with_gq=True):
        api.quantize_grad(dY, layout, self.N, self.C, self.H, self.W, params, self.s_state, has_prev,
                          self.gmax, self.stats, self.cls, self.vq, self.gq if with_gq else None,
                          seed, self.ws, sigma_override)
        torch.cuda.synchronize()
