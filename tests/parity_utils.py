"""Helpers shared by the GPU parity tests: tolerances and oracle / library adapters."""
import numpy as np
import torch

from oracle.gta_oracle import Shape as OracleShape

# Tolerances of the workload statement: bf16 storage with fp32 accumulation, and fp32.
BF16_REL_L2, BF16_MAX_ABS = 1e-2, 3e-2
F32_REL = 1e-4


def oracle_shape(w, seq=None, causal=1, scale=0.0):
    return OracleShape(w.batch, w.seq if seq is None else seq, w.d_model, w.n_heads, w.n_q, w.n_k, w.n_c,
                       w.d_h, w.d_l, causal, scale)


def cpu(t):
    return {k: (v.cpu() if isinstance(v, torch.Tensor) else v) for k, v in t.items()}


def assert_close(got, want, dtype, what=""):
    """got: torch tensor (any device); want: float64 numpy array from the oracle."""
    g = got.detach().to("cpu", torch.float64).numpy()
    assert g.shape == want.shape, (g.shape, want.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite output"
    err = g - want
    denom = np.sqrt((want ** 2).sum())
    rel_l2 = float(np.sqrt((err ** 2).sum()) / denom) if denom > 0 else float(np.abs(err).max())
    max_abs = float(np.abs(err).max()) if err.size else 0.0
    if dtype == torch.float32:
        scale = float(np.abs(want).max()) if want.size else 1.0
        assert rel_l2 <= F32_REL, f"{what}: rel-L2 {rel_l2:.3e} > {F32_REL}"
        assert max_abs <= F32_REL * max(scale, 1e-30), f"{what}: max-abs {max_abs:.3e} vs scale {scale:.3e}"
    else:
        assert rel_l2 <= BF16_REL_L2, f"{what}: rel-L2 {rel_l2:.3e} > {BF16_REL_L2}"
        assert max_abs <= BF16_MAX_ABS, f"{what}: max-abs {max_abs:.3e} > {BF16_MAX_ABS}"
    return rel_l2, max_abs
