"""Shared helpers of the GPU parity tests: bf16 bit patterns <-> torch tensors, tolerances."""
import numpy as np
import torch

from paper_2407_18121_b200 import workloads as wl

# Tolerances of the parity checks:
#   fp32 results (importance scores, lse): relative 1e-3
#   bf16 results (merged K/V rows, decode outputs): |gpu - oracle| <= 2e-2 + 2^-8 * |oracle|
#   (the relative term is bf16's own half-ulp bound, which exceeds 2e-2 once |x| >= 8)
SCORE_RTOL = 1e-3
BF16_ATOL = 2e-2
BF16_RTOL = 2.0 ** -8


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> CUDA bf16 tensor of the same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.view(torch.bfloat16).cuda()


def host_bits(t: torch.Tensor) -> np.ndarray:
    """CUDA/CPU bf16 tensor -> uint16 bit patterns."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)


def host_f64(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return wl.bf16_bits_to_f64(host_bits(t))
    return t.detach().cpu().double().numpy()


def assert_bf16_close(gpu: torch.Tensor, want: np.ndarray, what: str = ""):
    got = host_f64(gpu)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    bound = BF16_ATOL + BF16_RTOL * np.abs(want)
    bad = err > bound
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} elements out of tolerance; "
                           f"max abs err {err.max():.4g} at {np.unravel_index(err.argmax(), err.shape)}")


def assert_rel_close(gpu: torch.Tensor, want: np.ndarray, rtol: float, atol: float = 0.0, what: str = ""):
    got = host_f64(gpu)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    bound = atol + rtol * np.abs(want)
    bad = err > bound
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} out of tolerance; worst rel "
                           f"{(err / np.maximum(np.abs(want), 1e-300)).max():.4g}")


def scratch(nbytes: int) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device="cuda")


class Guarded:
    """A device buffer with poisoned guard bands on both sides, to catch out-of-bounds writes."""
    PAD = 256

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape))
        es = torch.empty((), dtype=dtype).element_size()
        self.raw = torch.full((2 * self.PAD + n * es,), 0xA5, dtype=torch.uint8, device="cuda")
        self.t = self.raw[self.PAD:self.PAD + n * es].view(dtype).view(*shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what=""):
        torch.cuda.synchronize()
        assert (self.raw[:self.PAD] == 0xA5).all().item(), f"{what}: write below the buffer"
        assert (self.raw[-self.PAD:] == 0xA5).all().item(), f"{what}: write past the buffer"
