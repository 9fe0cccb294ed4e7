"""Helpers shared by the GPU parity tests: move seeded inputs to the device, call the library
through its binding, and measure errors the way the tolerances are defined."""
import numpy as np

import wersa_inputs as wi


from wersa_inputs import device_inputs, to_device  # noqa: E402,F401  (re-exported for the tests)


def to_numpy64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def normalised_error(got, ref):
    """err = |got - ref| / max(|ref|, rms over the slab of ref); slabs are the leading two axes.
    Outputs of the operator are ~1/sqrt(n) the size of V with many near-zero entries, so a plain
    element-wise relative error is meaningless; errors are measured against the slab's rms."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    axes = tuple(range(2, ref.ndim)) if ref.ndim > 2 else None
    rms = np.sqrt(np.mean(ref ** 2, axis=axes, keepdims=True))
    denom = np.maximum(np.abs(ref), np.maximum(rms, 1e-300))
    return np.abs(got - ref) / denom


def small_vector_error(got, ref):
    """Scalars / small parameter vectors: |diff| / max(|ref|, 1e-12 + ||ref||_inf)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    scale = np.max(np.abs(ref)) if ref.size else 0.0
    return np.abs(got - ref) / max(scale, 1e-30)
