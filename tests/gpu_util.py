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


def check_attn(got_f64, want_f64):
    """The parity bar: max-abs <= 1e-2 and mean-abs <= 1e-3 against the fp64 oracle."""
    err = np.abs(got_f64 - want_f64)
    assert np.isfinite(got_f64).all()
    assert err.max() <= MAX_ABS, "max-abs error %.3e" % err.max()
    assert err.mean() <= MEAN_ABS, "mean-abs error %.3e" % err.mean()
    return err.max(), err.mean()


# Bounds of the two looser figures of the outlier workload (see check_attn_outliers).
OUTLIER_REL_MAX = 4e-2
OUTLIER_RAW_MAX = 100.0
OUTLIER_RAW_MEAN = 5e-2


def check_attn_outliers(got_f64, want_faithful, scale, want_truth, label=""):
    """The bars of the outlier workload (1 % of the entries x20), all three figures.

    The benchmark's absolute bar is stated for unit-variance inputs.  With
    entries of magnitude ~60 the cache *format* already breaks it: one bf16
    rounding of a rotated K or Q entry (half an ulp = 0.12) moves a score by
    ~0.5, whatever the kernel does.  So three figures are taken and printed:

    raw      |got - truth|, truth = the fp64 oracle on unrounded rotations.  It
             measures the format, not the kernel: where two outlier keys compete
             for a row, the rounding of the rotated K decides the winner and the
             output moves by the difference of their values (several units; a
             value can reach 20 x 5 sigma = 100, which is OUTLIER_RAW_MAX).  The
             mean is bounded by OUTLIER_RAW_MEAN so that a regression of an order of
             magnitude still fails.
    rel      |got - ref| / max(1, |ref|), ref = the oracle with rotated Q/K rounded
             to bf16 as the cache stores them.  Mean <= 1e-3; the maximum is
             bounded by OUTLIER_REL_MAX rather than 1e-2, because an output element can
             be a small difference of large terms: rounding the weights to bf16
             for the PV product and rounding the output each cost up to 2^-9 of
             sum_j p_j |v_j|, which |ref| does not see when the terms cancel.
    scaled   |got - ref| / max(1, sum_j p_j |v_j|), the magnitude of what an output
             element sums (``scale``, the oracle's attention over |V|).  This is the
             figure the 1e-2 / 1e-3 bar is applied to; for unit-variance inputs
             scale < 1 and it is the absolute bar itself.
    """
    assert np.isfinite(got_f64).all()
    raw = np.abs(got_f64 - want_truth)
    err = np.abs(got_f64 - want_faithful)
    rel = err / np.maximum(1.0, np.abs(want_faithful))
    scaled = err / np.maximum(1.0, scale)
    print("outliers %s: raw vs truth max %.3e mean %.3e | vs stored-format oracle: abs max %.3e mean %.3e, "
          "/max(1,|ref|) max %.3e mean %.3e, /max(1,sum p|v|) max %.3e mean %.3e"
          % (label, raw.max(), raw.mean(), err.max(), err.mean(), rel.max(), rel.mean(), scaled.max(), scaled.mean()))
    assert scaled.max() <= MAX_ABS, "scaled max error %.3e" % scaled.max()
    assert scaled.mean() <= MEAN_ABS, "scaled mean error %.3e" % scaled.mean()
    assert rel.mean() <= MEAN_ABS, "mean error relative to max(1, |ref|) %.3e" % rel.mean()
    assert rel.max() <= OUTLIER_REL_MAX, "max error relative to max(1, |ref|) %.3e" % rel.max()
    assert raw.max() <= OUTLIER_RAW_MAX and raw.mean() <= OUTLIER_RAW_MEAN, (raw.max(), raw.mean())
    return scaled.max(), scaled.mean()


def guarded(shape, dtype=None, fill=None, guard_rows=8):
    """A device tensor of ``shape`` with ``guard_rows`` extra leading-dimension rows
    before and after it, all filled with a pattern; returns (view, check) where
    check() asserts that the rows around the view still hold the pattern.  Stands in
    for a memory checker: a kernel that writes outside its rows trips it."""
    dtype = dtype or torch.bfloat16
    pattern = -1234.0
    full = torch.full((shape[0] + 2 * guard_rows,) + tuple(shape[1:]), pattern, device="cuda", dtype=dtype)
    view = full[guard_rows:guard_rows + shape[0]]
    if fill is not None:
        view.fill_(fill)

    def check():
        assert bool((full[:guard_rows] == pattern).all()), "rows before the tensor were written"
        assert bool((full[guard_rows + shape[0]:] == pattern).all()), "rows after the tensor were written"
    return view, check


def new_cache(wl, layers=None):
    return B.Cache(layers or wl.layers, wl.heads, wl.head_dim, wl.tokens_per_frame, wl.chunk_frames,
                   wl.sink_frames, wl.window_frames)
