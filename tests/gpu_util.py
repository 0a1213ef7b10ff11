"""Helpers shared by the GPU parity tests: tensor marshalling and tolerances."""
import numpy as np
import torch

from paper_2509_22622_b200 import binding as B
from paper_2509_22622_b200 import synth

# Tolerances of the benchmark definition for bf16 I/O on unit-variance inputs,
# against the fp64 oracle.
MAX_ABS = 1e-2
MEAN_ABS = 1e-3


def dev(bits: np.ndarray) -> torch.Tensor:
    """bf16 bit patterns (uint16) -> cuda bfloat16 tensor holding the same bytes."""
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)


def bits(t: torch.Tensor) -> np.ndarray:
    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def f64(t: torch.Tensor) -> np.ndarray:
    return synth.bf16_bits_to_f64(bits(t))


def ulp_distance(a_bits: np.ndarray, b_bits: np.ndarray) -> np.ndarray:
    """Distance in bf16 units-in-the-last-place between two bit-pattern arrays."""
    def key(u):
        u = u.astype(np.int32)
        return np.where(u & 0x8000, 0x8000 - u, u)      # sign-magnitude -> monotone integers
    return np.abs(key(a_bits) - key(b_bits))


def check_attn(got_f64, want_f64, scale=None):
    """The parity bar: max-abs <= 1e-2 and mean-abs <= 1e-3 against the oracle.

    ``scale`` is used by the outlier workload only.  It is sum_j p_j |v_j| (the
    oracle's attention over |V|), the magnitude of what each output element
    sums: rounding P to bf16 for the PV product and rounding the output to bf16
    each cost at most 2^-9 of it, so the error is measured in units of
    max(1, scale).  For unit-variance inputs scale < 1 and this is the absolute
    bar itself."""
    err = np.abs(got_f64 - want_f64)
    if scale is not None:
        err = err / np.maximum(1.0, scale)
    assert np.isfinite(got_f64).all()
    assert err.max() <= MAX_ABS, "max-abs error %.3e" % err.max()
    assert err.mean() <= MEAN_ABS, "mean-abs error %.3e" % err.mean()
    return err.max(), err.mean()


def new_cache(wl, layers=None):
    return B.Cache(layers or wl.layers, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames,
                   wl.sink_frames, wl.window_frames)
