"""Shared helpers for the GPU parity tests (host <-> device shuttling and the error bound)."""
import numpy as np
import torch

import oracle
from paper_2609_34380_b200 import workloads

# Parity bound for GEMM outputs against the FP64 oracle on the same effective weights.
REL_BOUND = 1e-2
# What the arithmetic actually allows: exact FP16 products, FP32 accumulation over K <= 28672
# (relative error of a sum of K terms <= K * 2^-24 of the sum of magnitudes, typically far
# less) and one FP16 rounding (2^-11 relative).  Checked as a tighter, second bound.
TIGHT_BOUND = 2e-3


def to_np_words(t: torch.Tensor) -> np.ndarray:
    return workloads.as_words(t)


def to_np_bytes(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().contiguous().numpy()


def y_as_f64(y: torch.Tensor) -> np.ndarray:
    return y.detach().cpu().to(torch.float64).numpy()


def assert_close_to_oracle(y_gpu, y_ref: np.ndarray, what=""):
    got = y_as_f64(y_gpu) if isinstance(y_gpu, torch.Tensor) else np.asarray(y_gpu, np.float64)
    scale = np.max(np.abs(y_ref))
    err = np.max(np.abs(got - y_ref)) if y_ref.size else 0.0
    assert np.all(np.isfinite(got)), what
    assert err <= REL_BOUND * scale, f"{what}: max err {err:.3e} > {REL_BOUND} * {scale:.3e}"
    assert err <= TIGHT_BOUND * scale, f"{what}: max err {err:.3e} > tight {TIGHT_BOUND} * {scale:.3e}"
    return err / scale if scale else 0.0


def split_both(w: torch.Tensor, enc_req: int, device="cuda:0", p_out=None, r_out=None):
    """Planes for the GPU (from dps_split_weights) and, independently, the oracle's planes of the same FP16
    words for the reference side of a parity test: the two paths meet only at their inputs.
    Returns (p, r, enc, p_ref, r_ref)."""
    import paper_2609_34380_b200 as dps
    p, r, enc = dps.dps_split_weights(w.to(device), enc_req, p_out, r_out)
    p_ref, r_ref, enc_ref = oracle.split(to_np_words(w), enc_req)
    assert enc == enc_ref, (enc, enc_ref)
    return p, r, enc, p_ref, r_ref


def split_on_host(w: torch.Tensor, enc: int):
    """Oracle split of a (possibly device) FP16 tensor -> numpy planes."""
    return oracle.split(to_np_words(w), enc)
