"""Helpers shared by the GPU parity tests (tensor upload, tolerance check)."""
import numpy as np
import torch

import synth

DEV = "cuda:0"


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 CUDA tensor of the same shape."""
    return torch.from_numpy(bits.view(np.int16).copy()).to(DEV).view(torch.bfloat16)


def host_f64_of_bf16(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def dev(a: np.ndarray) -> torch.Tensor:
    if a.dtype == np.uint64:
        return torch.from_numpy(a.view(np.int64).copy()).to(DEV)
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def host_u64(t: torch.Tensor) -> np.ndarray:
    return t.cpu().numpy().view(np.uint64)


def f64(bits: np.ndarray) -> np.ndarray:
    return synth.bf16_bits_to_f32(bits).astype(np.float64)


def assert_attention_close(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """bf16 attention outputs vs the fp64 oracle on the same bf16-rounded inputs:
    max |g - r| <= 2e-2 and ||g - r||_F / ||r||_F <= 1e-2."""
    got = got.astype(np.float64)
    err = np.abs(got - ref)
    rel = np.linalg.norm(got - ref) / max(np.linalg.norm(ref), 1e-30)
    assert err.max() <= 2e-2, f"{what}: max abs err {err.max():.4g} at {np.unravel_index(err.argmax(), err.shape)}"
    assert rel <= 1e-2, f"{what}: relative Frobenius err {rel:.4g}"


def assert_log_probs_close(got: np.ndarray, ref: np.ndarray, what: str = ""):
    """Log-probabilities of the bf16 decoder vs the fp64 oracle (rows of live beams only).

    A bf16 rounding of an activation is a relative error of at most u = 2^-9; after the roundings along the
    path the final hidden vector carries a relative rms error of a few u, and a logit z = h . w inherits it as
    (a few u) * std(z) rms.  The bound therefore scales with the spread of the row's logits:
        rms error <= 1.0e-2 * std   (about 5 u),      max error <= 5e-2 * std
    (the maximum of 1e7..1e8 near-normal errors sits about six rms above zero).  Measured worst cases:
    rms 0.0075 * std, max 0.04 * std (bf16 residual stream at the paper's decoder shape); the bound is that
    plus a margin and is not to be widened to make a test pass."""
    got, ref = got.astype(np.float64), ref.astype(np.float64)
    std = float(ref.std())
    err = np.abs(got - ref)
    rms = float(np.sqrt((err ** 2).mean()))
    assert err.max() <= 5e-2 * std, f"{what}: max log-prob error {err.max():.4g} at logit spread {std:.3g}"
    assert rms <= 1.0e-2 * std, f"{what}: rms log-prob error {rms:.4g} at logit spread {std:.3g}"


def assert_gemm_close(got: np.ndarray, ref: np.ndarray, abs_sum: np.ndarray, bf16_roundings: int, what: str = ""):
    """Element-wise bound for y = x w^T (+ epilogue) computed with bf16 operands and fp32 accumulation.

    abs_sum[m, n] = sum_k |x[m, k]| |w[n, k]| (+ |residual|): the scale of the accumulation error.  An fp32
    accumulation of K products, in whatever order the tensor core takes them, errs by a few ulps of that
    sum: allowed 2^-19 * abs_sum (2 ulps of fp32 at the size of the absolute sum).  Every rounding of the
    result to bf16 (output conversion; the bf16 add into a bf16 residual stream is a second one) adds at
    most 2^-9 of the value it rounds; allowed 2^-8 * |ref| per rounding.  Nothing scales with the largest
    element of the matrix: a dropped k-block or a mis-rounded epilogue of small magnitude fails."""
    got, ref = got.astype(np.float64), ref.astype(np.float64)
    bound = 2.0 ** -19 * abs_sum + bf16_roundings * 2.0 ** -8 * np.abs(ref) + 1e-30
    ratio = np.abs(got - ref) / bound
    i = np.unravel_index(ratio.argmax(), ratio.shape)
    assert ratio.max() <= 1.0, (f"{what}: |err| {abs(got[i] - ref[i]):.4g} at {i} is {ratio.max():.2f} x the bound "
                                f"(ref {ref[i]:.4g}, abs-sum {abs_sum[i]:.4g})")
