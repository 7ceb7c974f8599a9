"""Shared helpers for the parity tests (no attention arithmetic here)."""
import numpy as np

MAX_ABS = 1e-2     # bf16 in/out, fp32 accumulation: bound on any element
MEAN_ABS = 1e-3    # and on the mean absolute error


def bits_to_f64(bits: np.ndarray) -> np.ndarray:
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def pool_rows(pool_bits: np.ndarray) -> np.ndarray:
    """Undo the documented row layout of a KV pool [pages, Hkv, P, d]: the library stores the
    16-byte piece j of the row in slot r at position (j & ~7) | ((j & 7) ^ (r & 7))."""
    pages, hkv, P, d = pool_bits.shape
    pieces = pool_bits.reshape(pages, hkv, P, d // 8, 8)
    out = np.empty_like(pieces)
    for r in range(P):
        j = np.arange(d // 8)
        out[:, :, r, j] = pieces[:, :, r, (j & ~7) | ((j & 7) ^ (r & 7))]
    return out.reshape(pages, hkv, P, d)


def assert_attention_close(got_bits: np.ndarray, want: np.ndarray, what: str = "", allow_big: bool = True) -> int:
    """GPU bf16 output vs the unrounded fp64 oracle.

    The gate is max-abs 1e-2 and mean-abs 1e-3.  A bf16 result cannot be closer
    than half an ulp to the exact value, and for |O| >= 4 half an ulp (2^-7 and
    up) already exceeds 1e-2; only for such elements the bound is widened by
    that half ulp.  Returns how many elements needed that allowance (error above
    1e-2, within 1e-2 plus the half ulp), and with `allow_big=False` (the
    full-size configurations with their committed seeds) any such element fails
    the test, so that a seed which needs the allowance is a visible decision and
    not a silent one.
    """
    got = bits_to_f64(got_bits)
    assert got.shape == want.shape, (got.shape, want.shape)
    assert np.isfinite(got).all(), f"{what}: non-finite output"
    err = np.abs(got - want)
    mag = np.abs(want)
    half_ulp = np.where(mag >= 4.0, 2.0 ** (np.floor(np.log2(np.maximum(mag, 1e-30))) - 8), 0.0)
    big = int(((err > MAX_ABS) & (err <= MAX_ABS + half_ulp)).sum())
    if big:
        print(f"{what}: {big} elements with |O| >= 4 passed only with the half-ulp allowance")
    assert allow_big or big == 0, f"{what}: {big} elements with |O| >= 4 needed the half-ulp allowance"
    worst = int(np.argmax(err - half_ulp))
    assert (err <= MAX_ABS + half_ulp).all(), (
        f"{what}: max-abs {err.flat[worst]:.4g} at flat index {worst} "
        f"(got {got.flat[worst]:.6g}, want {want.flat[worst]:.6g})")
    assert err.mean() <= MEAN_ABS, f"{what}: mean-abs {err.mean():.4g}"
    return big
