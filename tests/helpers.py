"""Test-side utilities: bf16 bit handling written independently of both the oracle and the library."""
import numpy as np


def to_bf16_bits(x) -> np.ndarray:
    """float -> bf16 bit patterns, round to nearest even, in numpy integer arithmetic."""
    u = np.ascontiguousarray(np.asarray(x, dtype=np.float32)).view(np.uint32).astype(np.uint64)
    lsb = (u >> 16) & 1
    r = ((u + 0x7FFF + lsb) >> 16).astype(np.uint16)
    nan = (u & 0x7FFFFFFF) > 0x7F800000
    r[nan] = ((u[nan] >> 16) | 0x40).astype(np.uint16)
    return r


def from_bf16_bits(b) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def ordered(b) -> np.ndarray:
    """Order-preserving integer image of bf16 bit patterns (+0 and -0 coincide)."""
    b = np.asarray(b, dtype=np.uint16).astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def ulp_distance(a, b) -> np.ndarray:
    return np.abs(ordered(a) - ordered(b))


def within_tol(got_bits, want_bits, atol=2e-2, rtol=2e-2):
    g = from_bf16_bits(got_bits).astype(np.float64)
    w = from_bf16_bits(want_bits).astype(np.float64)
    return np.abs(g - w) <= atol + rtol * np.abs(w)


def assert_close_bits(got_bits, want_bits, atol=2e-2, rtol=2e-2, what=""):
    ok = within_tol(got_bits, want_bits, atol, rtol)
    if not ok.all():
        g = from_bf16_bits(got_bits).astype(np.float64)
        w = from_bf16_bits(want_bits).astype(np.float64)
        bad = np.argwhere(~ok)
        i = tuple(bad[0])
        raise AssertionError(f"{what}: {len(bad)} of {ok.size} elements outside |d| <= {atol}+{rtol}|ref|; "
                             f"first at {i}: got {g[i]}, want {w[i]}; max abs err {np.abs(g - w).max()}")
