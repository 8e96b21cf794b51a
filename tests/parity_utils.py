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


class Guarded:
    """A device buffer between two guard bands (a page of 0xA5 bytes before and after it): a store that
    strays past either end of an output or a workspace shows up in check()."""
    GUARD = 4096

    def __init__(self, shape, dtype, device="cuda", fill_byte=0xFF):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = n
        self.raw = torch.full((2 * self.GUARD + ((n + 255) & ~255),), 0xA5, dtype=torch.uint8, device=device)
        body = self.raw[self.GUARD:self.GUARD + n]
        body.fill_(fill_byte)                    # NaN bit patterns for the floating-point types
        self.t = body.view(dtype).view(shape)

    def check(self, what=""):
        g = self.GUARD
        assert bool((self.raw[:g] == 0xA5).all()), f"{what}: bytes before the buffer were overwritten"
        assert bool((self.raw[g + self.nbytes:] == 0xA5).all()), f"{what}: bytes behind the buffer were overwritten"
