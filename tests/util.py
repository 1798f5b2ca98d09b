"""Helpers shared by the GPU parity tests: oracle-side quantisation -> device tensors and comparisons."""
from __future__ import annotations

import numpy as np
import torch

from oracle import formats as F

TORCH_OF = {"f32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16,
            "e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}


def to_device(x: np.ndarray, fmt: str, ld: int | None = None) -> torch.Tensor:
    """Round float32 host data to `fmt` with the oracle's quantiser and upload the bit patterns.

    With ld > cols the tensor is a view into a padded allocation (row pitch ld elements)."""
    x = np.ascontiguousarray(x)
    if fmt == "f32":
        t = torch.from_numpy(x.astype(np.float32))
    else:
        codes = F.quantise_codes(x, F.FORMATS[fmt])
        if codes.dtype == np.uint16:
            t = torch.from_numpy(codes.view(np.int16)).view(TORCH_OF[fmt])
        else:
            t = torch.from_numpy(codes).view(TORCH_OF[fmt])
    t = t.cuda()
    if ld is not None and ld != x.shape[1]:
        buf = torch.zeros((x.shape[0], ld), dtype=torch.uint8 if t.element_size() == 1 else t.dtype, device="cuda")
        buf = buf.view(t.dtype) if t.element_size() == 1 else buf
        buf[:, : x.shape[1]] = t
        t = buf[:, : x.shape[1]]
    return t


def values_of(x: np.ndarray, fmt: str) -> np.ndarray:
    """The float64 values the device tensor made by to_device holds."""
    if fmt == "f32":
        return x.astype(np.float32).astype(np.float64)
    return F.quantise(x, F.FORMATS[fmt])


def empty(rows: int, cols: int, fmt: str, ld: int | None = None) -> torch.Tensor:
    ld = ld or cols
    buf = torch.zeros((rows, ld), dtype=TORCH_OF[fmt], device="cuda") if TORCH_OF[fmt].itemsize > 1 else \
        torch.zeros((rows, ld), dtype=torch.uint8, device="cuda").view(TORCH_OF[fmt])
    return buf[:, :cols]


def codes_of(t: torch.Tensor) -> np.ndarray:
    t = t.contiguous()
    if t.element_size() == 1:
        return t.view(torch.uint8).cpu().numpy()
    if t.element_size() == 2:
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    raise ValueError(t.dtype)


def host_values(t: torch.Tensor) -> np.ndarray:
    return t.to(torch.float64).cpu().numpy() if t.element_size() > 1 else \
        t.contiguous().to(torch.float32).to(torch.float64).cpu().numpy()


def code_distance(got_codes: np.ndarray, want_codes: np.ndarray, fmt: str) -> np.ndarray:
    """|difference| of sign-magnitude codes read as integers on a common number line."""
    bits = F.FORMATS[fmt].bits
    sign = 1 << (bits - 1)

    def line(c):
        c = c.astype(np.int64)
        return np.where(c & sign, -(c & (sign - 1)), c & (sign - 1))

    return np.abs(line(got_codes) - line(want_codes))


def ulp_of(ref: np.ndarray, fmt: str) -> np.ndarray:
    """Spacing of `fmt` around each reference value."""
    f = F.FORMATS[fmt]
    a = np.abs(ref)
    _, ex = np.frexp(np.where(a > 0, a, 1.0))
    e = np.maximum(ex - 1, f.min_exp)
    return np.ldexp(1.0, e - f.M)


def code_deltas(got: torch.Tensor, want_codes: np.ndarray, fmt: str, extra=0.0, max_flip_fraction: float = 2e-3):
    """FP8 output check.  Every stored code must be within one step of the oracle's code, or -- where
    `extra` (an element-wise value-space allowance derived from a legitimate upstream rounding flip)
    is non-zero -- within one format spacing plus that allowance in value.  Differences must be rare.
    Returns (device value - oracle value) per element (zero except at those places)."""
    f = F.FORMATS[fmt]
    gc = codes_of(got)
    d = code_distance(gc, want_codes, fmt)
    delta = F.decode(gc, f) - F.decode(want_codes, f)
    ref = F.decode(want_codes, f)
    ok = (d <= 1) | (np.abs(delta) <= ulp_of(ref, fmt) + extra)
    assert ok.all(), f"FP8 output off by more than one step at {(~ok).sum()} places, worst code distance {d[~ok].max()}"
    assert (d > 0).mean() <= max_flip_fraction, f"flip fraction {(d > 0).mean():.2e}"
    return delta


def propagated(a: np.ndarray, b: np.ndarray, sparse_side: str) -> np.ndarray:
    """|a| @ |b|, where the operand named by sparse_side ("a" or "b") is a sparse matrix of rare
    upstream rounding flips: an element-wise bound on how far they can move a downstream matmul."""
    from scipy import sparse
    if sparse_side == "a":
        return np.asarray(sparse.csr_matrix(np.abs(a)) @ np.abs(b))
    return np.asarray((sparse.csr_matrix(np.abs(b).T) @ np.abs(a).T).T)


def assert_close_stored(got: torch.Tensor, ref: np.ndarray, fmt: str, abs_tol, what: str = ""):
    """Output-vs-oracle check for one stored tensor.

    f32: |d| <= abs_tol.  16-bit: |d| <= abs_tol + 1 ulp of the format at the reference.
    FP8: codes within one step of q(ref), except where ref is within abs_tol of the
    rounding boundary two steps away (not needed in practice, kept strict)."""
    g = host_values(got)
    if fmt == "f32":
        err = np.abs(g - ref)
        assert np.all(err <= abs_tol), f"{what}: max abs err {err.max():.3e} > {abs_tol:.1e}"
    elif fmt in ("bf16", "fp16"):
        err = np.abs(g - ref)
        lim = abs_tol + ulp_of(ref, fmt)
        bad = err > lim
        assert not bad.any(), f"{what}: {bad.sum()} elements beyond 1 ulp, worst {err[bad].max():.3e}"
    else:
        want = F.quantise_codes(ref, F.FORMATS[fmt])
        d = code_distance(codes_of(got), want, fmt)
        assert d.max() <= 1, f"{what}: FP8 code distance {d.max()} (count {(d > 1).sum()})"
