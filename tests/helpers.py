"""Shared helpers of the GPU parity tests (tensor conversion, tolerances)."""
import numpy as np
import torch

# attention output: bf16 inputs, fp32 accumulation, bf16 result
O_ATOL, O_RTOL = 1e-2, 2e-2
# attention mass, lse-derived probabilities, vocab probabilities
P_RTOL = 1e-4


def bf16_cuda(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def bits_of(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().view(torch.int16).numpy().view(np.uint16)


def assert_o_close(o_gpu: torch.Tensor, o_ref: np.ndarray):
    got = bf16_to_f64(o_gpu)
    err = np.abs(got - o_ref)
    bound = O_ATOL + O_RTOL * np.abs(o_ref)
    assert (err <= bound).all(), f"O mismatch: max err {err.max():.3e}, worst ratio {(err / bound).max():.3f}"
    return float((err / bound).max())


def assert_rel_close(got: np.ndarray, ref: np.ndarray, rtol=P_RTOL, what="value"):
    got = np.asarray(got, dtype=np.float64)
    err = np.abs(got - ref)
    bound = rtol * np.abs(ref) + 1e-30
    assert (err <= bound).all(), f"{what} mismatch: worst rel err {(err / (np.abs(ref) + 1e-300)).max():.3e}"
    return float((err / (np.abs(ref) + 1e-300)).max())
