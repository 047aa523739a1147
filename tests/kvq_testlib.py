"""Helpers shared by the GPU parity tests: run the same seeded problem through the CUDA
library (via the C ABI binding) and through the CPU oracle."""
import math

import numpy as np
import torch

from oracle import kvq_oracle as O
from paper_2605_26266_b200 import inputs

REL_L2_TOL = 1e-2      # attention output, relative L2 against the oracle
MAX_ABS_TOL = 2e-2     # attention output, largest absolute deviation


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """BF16 bit patterns (uint16) -> torch.bfloat16 CUDA tensor with the same bits."""
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def from_dev_bf16(t: torch.Tensor) -> np.ndarray:
    """torch.bfloat16 tensor -> float64 numpy."""
    return O.bf16_bits_to_f64(t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16))


def gpu_cache_arrays(cache, n):
    """The GPU cache's first n tokens as numpy arrays named like the oracle's."""
    v = cache.views()
    out = {}
    for name, t in v.items():
        a = t[:, :, :n].cpu().numpy()
        out[name] = a.view(np.uint16) if "zero" in name else a
    return out


def assert_cache_equal(gpu, oracle_cache, n, units=None):
    """Bit-exact comparison of packed codes, scale bytes and zero-point bits."""
    for name in ("k_codes", "v_codes", "k_scale", "v_scale", "k_zero", "v_zero"):
        g = gpu[name]
        o = getattr(oracle_cache, name)[:, :, :n]
        if units is not None:
            g = np.stack([g[b, h] for (b, h) in units])[None]
        assert g.shape == o.shape, (name, g.shape, o.shape)
        bad = int((g != o).sum())
        assert bad == 0, f"{name}: {bad} of {g.size} bytes differ"


def attn_errors(got: np.ndarray, want: np.ndarray):
    rel = float(np.linalg.norm(got - want) / max(np.linalg.norm(want), 1e-30))
    mx = float(np.abs(got - want).max())
    return rel, mx


def assert_attn_close(got, want, what=""):
    rel, mx = attn_errors(got, want)
    assert rel <= REL_L2_TOL and mx <= MAX_ABS_TOL, f"{what}: rel-L2 {rel:.3e}, max-abs {mx:.3e}"
    return rel, mx


def sigma_of(d):
    return 1.0 / math.sqrt(d)
