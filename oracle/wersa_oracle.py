"""ctypes binding of the float64 CPU oracle (oracle/wersa_oracle.cpp).

TEST INFRASTRUCTURE, NOT PRODUCT CODE: only tests/, the smoke check and the
benchmark's CPU-baseline leg may import this module.  It never touches CUDA and
shares nothing with the CUDA library.

`build()` compiles the C++ file with g++ (-O2 -fopenmp) into
oracle/libwersa_oracle.so; every wrapper below builds it on first use.
"""
import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wersa_oracle.cpp")
_LIB = os.path.join(_HERE, "libwersa_oracle.so")

_c_double_p = ctypes.POINTER(ctypes.c_double)
_c_int_p = ctypes.POINTER(ctypes.c_int)


def build(force=False):
    """Compile the oracle if the shared object is missing or older than its source."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    cmd = ["g++", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c++17", "-o", _LIB, _SRC]
    subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _dp(a):
    return None if a is None else a.ctypes.data_as(_c_double_p)


def _f64(a):
    """Contiguous float64 copy of an input; widening float32 (or bf16-valued float32) is exact."""
    if a is None:
        return None
    return np.ascontiguousarray(a, dtype=np.float64)


def threads():
    return int(_load().wersa_oracle_threads())


def next_pow2(n):
    p = 1
    while p < n:
        p <<= 1
    return p


def dwt(x, L):
    """Literal Haar analysis (Algorithm 2, Eqs. 19-20) of x (n, d).

    Returns the coefficient list [d_1, ..., d_L, a_L]; n is zero-padded to a power of two."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    n, d = x.shape
    npad = next_pow2(n)
    flat = np.zeros(npad * d, dtype=np.float64)
    rc = _load().wersa_oracle_dwt(_dp(x), n, d, L, _dp(flat))
    if rc:
        raise ValueError("oracle dwt: bad arguments")
    out, off = [], 0
    for i in range(L + 1):
        rows = npad >> (i + 1) if i < L else npad >> L
        out.append(flat[off:off + rows * d].reshape(rows, d).copy())
        off += rows * d
    return out


def idwt(coeffs):
    """Literal Haar synthesis (Algorithm 2, Eqs. 21-22) from [d_1, ..., d_L, a_L]."""
    L = len(coeffs) - 1
    d = coeffs[0].shape[1]
    npad = coeffs[0].shape[0] * 2
    flat = np.ascontiguousarray(np.concatenate([np.asarray(c, dtype=np.float64).reshape(-1)
                                                for c in coeffs]))
    x = np.zeros((npad, d), dtype=np.float64)
    rc = _load().wersa_oracle_idwt(_dp(flat), npad, d, L, _dp(x))
    if rc:
        raise ValueError("oracle idwt: bad arguments")
    return x


def haar_filter(x, f):
    """trim(IDWT(f (.) DWT(pad(x)))) for x (n, d), f (L+1,) ordered d_1..d_L, a_L."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    f = np.ascontiguousarray(f, dtype=np.float64)
    n, d = x.shape
    out = np.zeros_like(x)
    rc = _load().wersa_oracle_filter(_dp(x), n, d, len(f) - 1, _dp(f), _dp(out))
    if rc:
        raise ValueError("oracle filter: bad arguments")
    return out


def features(x, W, beta=1.0, bw_floor=1e-6):
    """phi(x) = ReLU(x W / max(beta, floor)) / sqrt(m), rows of x (n, d), W (d, m)."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    W = np.ascontiguousarray(W, dtype=np.float64)
    n, d = x.shape
    m = W.shape[1]
    phi = np.zeros((n, m), dtype=np.float64)
    _load().wersa_oracle_features(_dp(x), n, d, m, _dp(W), ctypes.c_double(float(beta)),
                                  ctypes.c_double(float(bw_floor)), _dp(phi))
    return phi


def gate(Q, gate_w, gate_b, omega, L, gate_per_head=1):
    """Mean-pooled query and per-scale filter (Eqs. 1-3). Q (B,H,n,d). Returns (qbar, f)."""
    Q = _f64(Q)
    B, H, n, d = Q.shape
    gw, gb, om = _f64(gate_w), _f64(gate_b), _f64(omega)
    qbar = np.zeros((B, H, d), dtype=np.float64)
    f = np.zeros((B, H, L + 1), dtype=np.float64)
    lib = _load()
    lib.wersa_oracle_gate(B, H, n, d, L, int(gate_per_head), _dp(Q), _dp(gw), _dp(gb), _dp(om),
                          _dp(qbar), _dp(f))
    return qbar, f


def forward(Q, K, V, W, beta, gate_w, gate_b, omega, L, eps=1e-6, bw_floor=1e-6,
            gate_per_head=1, sample_rows=None, want_aux=False):
    """Whole WERSA forward in float64.

    Q, K, V: (B,H,n,d); W: (d,m); gate_w: (H,d,L+1) or None; gate_b: (H,L+1) or None;
    omega: (L+1,).  Returns O (B,H,n,d) float64, or (O, aux) with aux = dict(f, qbar, S, z, D).
    With sample_rows (1-D int array) only those query rows are computed; other rows are NaN."""
    Q, K, V, W = _f64(Q), _f64(K), _f64(V), _f64(W)
    B, H, n, d = Q.shape
    m = W.shape[1]
    gw, gb, om = _f64(gate_w), _f64(gate_b), _f64(omega)
    O = np.full((B, H, n, d), np.nan, dtype=np.float64)
    f = np.zeros((B, H, L + 1), dtype=np.float64)
    qbar = np.zeros((B, H, d), dtype=np.float64)
    S = np.zeros((B, H, m, d), dtype=np.float64)
    z = np.zeros((B, H, m), dtype=np.float64)
    D = np.full((B, H, n), np.nan, dtype=np.float64)
    if sample_rows is not None:
        rows = np.ascontiguousarray(sample_rows, dtype=np.int32)
        rows_p, n_rows = rows.ctypes.data_as(_c_int_p), int(rows.size)
    else:
        rows_p, n_rows = None, 0
    lib = _load()
    rc = lib.wersa_oracle_forward(
        B, H, n, d, L, m, ctypes.c_double(eps), ctypes.c_double(bw_floor), int(gate_per_head),
        _dp(Q), _dp(K), _dp(V), _dp(W), ctypes.c_double(float(beta)), _dp(gw), _dp(gb), _dp(om),
        _dp(O), _dp(f), _dp(qbar), _dp(S), _dp(z), _dp(D), rows_p, n_rows)
    if rc:
        raise ValueError("oracle forward: bad arguments")
    if want_aux:
        return O, dict(f=f, qbar=qbar, S=S, z=z, D=D)
    return O


def backward(Q, K, V, W, beta, gate_w, gate_b, omega, dO, L, eps=1e-6, bw_floor=1e-6,
             gate_per_head=1):
    """Whole WERSA backward in float64 (chain rule through the forward steps).

    Returns dict(dQ, dK, dV, dbeta, dgate_w, dgate_b, domega, dbeta_closed)."""
    Q, K, V, W, dO = _f64(Q), _f64(K), _f64(V), _f64(W), _f64(dO)
    B, H, n, d = Q.shape
    m = W.shape[1]
    gw, gb, om = _f64(gate_w), _f64(gate_b), _f64(omega)
    dQ = np.zeros((B, H, n, d), dtype=np.float64)
    dK = np.zeros_like(dQ)
    dV = np.zeros_like(dQ)
    dbeta = np.zeros(1, dtype=np.float64)
    dbeta_closed = np.zeros(1, dtype=np.float64)
    dgw = np.zeros((H, d, L + 1), dtype=np.float64)
    dgb = np.zeros((H, L + 1), dtype=np.float64)
    dom = np.zeros(L + 1, dtype=np.float64)
    lib = _load()
    rc = lib.wersa_oracle_backward(
        B, H, n, d, L, m, ctypes.c_double(eps), ctypes.c_double(bw_floor), int(gate_per_head),
        _dp(Q), _dp(K), _dp(V), _dp(W), ctypes.c_double(float(beta)), _dp(gw), _dp(gb), _dp(om),
        _dp(dO), _dp(dQ), _dp(dK), _dp(dV), _dp(dbeta), _dp(dgw), _dp(dgb), _dp(dom),
        _dp(dbeta_closed))
    if rc:
        raise ValueError("oracle backward: bad arguments")
    return dict(dQ=dQ, dK=dK, dV=dV, dbeta=float(dbeta[0]), dgate_w=dgw, dgate_b=dgb,
                domega=dom, dbeta_closed=float(dbeta_closed[0]))


if __name__ == "__main__":
    print(build(force=True))
