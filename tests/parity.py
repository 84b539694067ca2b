"""Shared helpers of the parity tests: tolerances and host<->device conversion."""
import numpy as np
import torch

# Tolerances of the CUDA path against the oracle on identical bf16-rounded inputs:
# relative Frobenius error <= 2e-3 and max |err| <= 1e-2 * max |ref| per tensor;
# 1e-6 relative (Frobenius) for the fp32 optimiser update.
REL_FRO = 2e-3
MAX_REL = 1e-2
SGD_REL = 1e-6


def dev_bf16(x: np.ndarray) -> torch.Tensor:
    """fp32/fp64 values already on the bf16 grid -> device bf16 tensor (exact)."""
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(torch.bfloat16).cuda().contiguous()


def dev_f32(x: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).cuda().contiguous()


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


def errors(got: np.ndarray, ref: np.ndarray):
    got = np.asarray(got, np.float64).reshape(-1)
    ref = np.asarray(ref, np.float64).reshape(-1)
    nref = np.linalg.norm(ref)
    rel = np.linalg.norm(got - ref) / nref if nref > 0 else np.linalg.norm(got)
    mx = np.max(np.abs(ref)) if ref.size else 0.0
    maxerr = np.max(np.abs(got - ref)) / mx if mx > 0 else np.max(np.abs(got), initial=0.0)
    return rel, maxerr


def assert_close(got, ref, name, rel_fro=REL_FRO, max_rel=MAX_REL):
    got = host(got) if isinstance(got, torch.Tensor) else np.asarray(got, np.float64)
    assert got.shape == tuple(np.shape(ref)), f"{name}: shape {got.shape} vs {np.shape(ref)}"
    assert np.all(np.isfinite(got)), f"{name}: non-finite values"
    rel, mx = errors(got, ref)
    assert rel <= rel_fro and mx <= max_rel, f"{name}: relF={rel:.3e} (<= {rel_fro}), max|err|/max|ref|={mx:.3e} (<= {max_rel})"
    return rel, mx
