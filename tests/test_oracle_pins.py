"""Pins of the float64 oracle to things other than itself: closed forms, invariants, a
hand-derived worked example, brute force, Monte-Carlo limits and finite differences.
Each test names the passage of the paper it pins.  CPU only."""
import math
import os

import numpy as np
import pytest

from oracle import wersa_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------- independent numpy helpers
def block_mean(x, size):
    """Mean over aligned blocks of `size` rows, broadcast back (zero-padded tail)."""
    n, d = x.shape
    npad = -(-n // size) * size
    xp = np.zeros((npad, d))
    xp[:n] = x
    mu = xp.reshape(npad // size, size, d).mean(axis=1)
    return np.repeat(mu, size, axis=0)[:n]


def filter_by_block_means(x, f):
    """T_f x = f_0 x + sum_{i=1..L} (f_i - f_{i-1}) blockmean_{2^i}(x): follows from the Haar
    detail-l projector being blockmean_{2^(l-1)} - blockmean_{2^l}."""
    out = f[0] * x
    for i in range(1, len(f)):
        out = out + (f[i] - f[i - 1]) * block_mean(x, 2 ** i)
    return out


def brute_force_attention(QF, KF, V, W, beta, eps, bw_floor=1e-6):
    """Quadratic form of Eq. 7: O_t = sum_j k(t,j) V_j / (sum_j k(t,j) + eps)."""
    m = W.shape[1]
    bw = max(beta, bw_floor)
    pq = np.maximum(QF @ W / bw, 0.0) / math.sqrt(m)
    pk = np.maximum(KF @ W / bw, 0.0) / math.sqrt(m)
    kern = pq @ pk.T                      # n x n
    return (kern @ V) / (kern.sum(axis=1, keepdims=True) + eps)


def read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            out[key] = np.array([float(v) for v in vals])
    return out


# ---------------------------------------------------------------- Haar analysis / synthesis
@pytest.mark.parametrize("n,d,L", [(8, 1, 3), (64, 5, 3), (256, 4, 8), (1024, 3, 5), (16, 2, 1)])
def test_perfect_reconstruction_and_energy(n, d, L):
    # Eqs. 19-22: orthonormal pair => IDWT(DWT(x)) = x and energy is preserved.
    rng = np.random.default_rng(n + L)
    x = rng.standard_normal((n, d))
    coeffs = orc.dwt(x, L)
    assert [c.shape[0] for c in coeffs] == [n >> (l + 1) for l in range(L)] + [n >> L]
    rec = orc.idwt(coeffs)
    assert np.max(np.abs(rec - x)) < 1e-12
    energy = sum(float((c ** 2).sum()) for c in coeffs)
    assert abs(energy - float((x ** 2).sum())) < 1e-10 * float((x ** 2).sum())


def test_worked_example_w1():
    g = read_golden("haar_w1.txt")
    x = g["x"].reshape(-1, 1)
    d1, d2, a2 = orc.dwt(x, 2)
    assert np.allclose(d1[:, 0], g["d1"], atol=1e-15)
    assert np.allclose(d2[:, 0], g["d2"], atol=1e-15)
    assert np.allclose(a2[:, 0], g["a2"], atol=1e-15)
    xf = orc.haar_filter(x, g["f"])
    assert np.allclose(xf[:, 0], g["x_F"], atol=1e-14)


def test_band_localisation_and_order():
    # Coefficient order [d_1..d_L, a_L] (Algorithm 2): a constant lives only in a_L,
    # an alternating +-c signal only in d_1, a period-4 square wave (++--) only in d_2.
    n, L = 32, 3
    const = np.full((n, 1), 3.0)
    alt = np.tile(np.array([[2.0], [-2.0]]), (n // 2, 1))
    sq = np.tile(np.array([[1.0], [1.0], [-1.0], [-1.0]]), (n // 4, 1))
    for sig, band in ((const, 3), (alt, 0), (sq, 1)):
        coeffs = orc.dwt(sig, L)
        for i, c in enumerate(coeffs):
            if i == band:
                assert np.abs(c).max() > 1.0
            else:
                assert np.abs(c).max() < 1e-12
    # sign convention d = (even - odd)/sqrt2: a step down gives a positive detail.
    step = np.array([[1.0], [0.0]])
    assert orc.dwt(step, 1)[0][0, 0] == pytest.approx(1 / math.sqrt(2))
    # hence the per-scale gate hits the right band
    f = np.array([0.25, 0.5, 0.75, 2.0])
    assert np.allclose(orc.haar_filter(const, f), 2.0 * const)
    assert np.allclose(orc.haar_filter(alt, f), 0.25 * alt)
    assert np.allclose(orc.haar_filter(sq, f), 0.5 * sq)


@pytest.mark.parametrize("n,L", [(64, 3), (256, 8), (96, 4), (50, 3), (1000, 5)])
def test_filter_equals_block_mean_identity(n, L):
    rng = np.random.default_rng(7 * n + L)
    x = rng.standard_normal((n, 6)) + 0.3
    f = rng.uniform(0.1, 1.5, L + 1)
    got = orc.haar_filter(x, f)
    want = filter_by_block_means(x, f)
    assert np.max(np.abs(got - want)) < 1e-12


def test_filter_algebra():
    rng = np.random.default_rng(11)
    n, d, L = 64, 4, 4
    x, y = rng.standard_normal((n, d)), rng.standard_normal((n, d))
    f, g = rng.uniform(0.2, 1.2, L + 1), rng.uniform(0.2, 1.2, L + 1)
    # all gates equal => plain scaling
    assert np.allclose(orc.haar_filter(x, np.full(L + 1, 0.5)), 0.5 * x, atol=1e-13)
    # symmetric operator: <T_f x, y> = <x, T_f y>
    assert float((orc.haar_filter(x, f) * y).sum()) == pytest.approx(
        float((x * orc.haar_filter(y, f)).sum()), rel=1e-12)
    # composition multiplies gates band by band
    assert np.allclose(orc.haar_filter(orc.haar_filter(x, f), g), orc.haar_filter(x, f * g),
                       atol=1e-12)
    # linear in f
    assert np.allclose(orc.haar_filter(x, f) + orc.haar_filter(x, g), orc.haar_filter(x, f + g),
                       atol=1e-12)


def test_pad_and_trim_rule():
    # Algorithm 2 pads to the next power of two and trims; because L Haar levels only mix rows
    # inside aligned blocks of 2^L, padding to the next multiple of 2^L gives the same rows.
    rng = np.random.default_rng(5)
    n, d, L = 40, 3, 3                      # next pow2 = 64, next multiple of 8 = 40
    x = rng.standard_normal((n, d))
    f = rng.uniform(0.2, 1.2, L + 1)
    got = orc.haar_filter(x, f)
    n2 = 44                                 # not a multiple of 8: tail block is zero-filled
    x2 = rng.standard_normal((n2, d))
    got2 = orc.haar_filter(x2, f)
    xp = np.zeros((48, d))
    xp[:n2] = x2
    assert np.allclose(got, filter_by_block_means(x, f), atol=1e-13)
    assert np.allclose(got2, orc.haar_filter(xp, f)[:n2], atol=1e-13)


# ---------------------------------------------------------------- gate (Eqs. 1-3)
def test_gate_pins():
    rng = np.random.default_rng(3)
    B, H, n, d, L = 2, 3, 16, 4, 2
    Q = rng.standard_normal((B, H, n, d))
    gw = rng.standard_normal((H, d, L + 1)) * 0.3
    gb = rng.standard_normal((H, L + 1)) * 0.3
    om = rng.uniform(0.5, 1.5, L + 1)
    qbar, f = orc.gate(Q, None, gb, om, L)
    assert np.allclose(qbar, Q.mean(axis=2), atol=1e-14)
    sig = 1.0 / (1.0 + np.exp(-gb))
    assert np.allclose(f, np.broadcast_to(sig * om, (B, H, L + 1)), atol=1e-14)
    # shifting every query row by delta moves the logits by gate_w^T delta exactly
    delta = rng.standard_normal(d)
    _, f0 = orc.gate(Q, gw, gb, om, L)
    _, f1 = orc.gate(Q + delta, gw, gb, om, L)
    logit = lambda p: np.log(p / (1 - p))
    shift = logit(f1 / om) - logit(f0 / om)
    want = np.einsum("hci,c->hi", gw, delta)
    assert np.allclose(shift, np.broadcast_to(want, (B, H, L + 1)), atol=1e-11)
    # batch-wide gate of Algorithm 1: one linear map over the concatenated heads, bias row 0
    _, fb = orc.gate(Q, gw, gb, om, L, gate_per_head=0)
    pooled = Q.mean(axis=2).reshape(B, H * d)
    u = pooled @ gw.reshape(H * d, L + 1) + gb[0]
    want_f = om / (1.0 + np.exp(-u))
    assert np.allclose(fb, np.repeat(want_f[:, None, :], H, axis=1), atol=1e-13)


# ---------------------------------------------------------------- feature map (Eq. 6)
def arc_cosine_kernel(x, y):
    """E_w[ReLU(w.x) ReLU(w.y)], w ~ N(0, I): |x||y| (sin t + (pi - t) cos t) / (2 pi)."""
    nx, ny = np.linalg.norm(x), np.linalg.norm(y)
    t = math.acos(np.clip(x @ y / (nx * ny), -1, 1))
    return nx * ny * (math.sin(t) + (math.pi - t) * math.cos(t)) / (2 * math.pi)


def test_feature_map_monte_carlo_converges_to_arc_cosine_kernel():
    # phi(x).phi(y) is a Monte-Carlo estimate, error ~ C/sqrt(m) (Appendix B): with the 1/sqrt(m)
    # scaling of Algorithm 1 it converges to the ReLU-Gaussian kernel / bw^2.
    d, beta = 8, 1.7
    rng = np.random.default_rng(0)
    x, y = rng.standard_normal(d), rng.standard_normal(d)
    want = arc_cosine_kernel(x, y) / beta ** 2
    errs = {}
    for m in (2 ** 8, 2 ** 12, 2 ** 16):
        est = []
        for rep in range(12):
            W = np.random.default_rng(1000 * m + rep).standard_normal((d, m))
            phi = orc.features(np.stack([x, y]), W, beta=beta)
            assert phi.min() >= 0.0
            est.append(float(phi[0] @ phi[1]))
        errs[m] = float(np.sqrt(np.mean((np.array(est) - want) ** 2)))
    assert errs[2 ** 16] < 0.02 * abs(want)
    # rate: 16x more features => ~4x smaller rms error (allow a factor 2 of slack on 12 reps)
    assert errs[2 ** 12] < errs[2 ** 8] / 2.0
    assert errs[2 ** 16] < errs[2 ** 12] / 2.0


def test_feature_map_homogeneity_and_floor():
    rng = np.random.default_rng(4)
    x, W = rng.standard_normal((5, 6)), rng.standard_normal((6, 32))
    p1 = orc.features(x, W, beta=1.0)
    assert np.allclose(orc.features(x, W, beta=2.5), p1 / 2.5, atol=1e-14)
    assert np.allclose(p1, np.maximum(x @ W, 0) / math.sqrt(32), atol=1e-13)
    # bw = max(beta, floor)
    assert np.allclose(orc.features(x, W, beta=-3.0, bw_floor=0.5), p1 / 0.5, atol=1e-13)


# ---------------------------------------------------------------- whole forward (Eq. 7)
def small_problem(seed, B=2, H=2, n=48, d=8, L=3, m=16, gates=True):
    rng = np.random.default_rng(seed)
    p = dict(Q=rng.standard_normal((B, H, n, d)) + 0.2, K=rng.standard_normal((B, H, n, d)),
             V=rng.standard_normal((B, H, n, d)), W=rng.standard_normal((d, m)),
             omega=rng.uniform(0.5, 1.5, L + 1))
    p["gate_w"] = rng.standard_normal((H, d, L + 1)) * 0.5 if gates else None
    p["gate_b"] = rng.standard_normal((H, L + 1)) * 0.5 if gates else None
    return p


@pytest.mark.parametrize("n,per_head", [(64, 1), (48, 1), (37, 0)])
def test_forward_matches_brute_force_quadratic_attention(n, per_head):
    L, beta, eps = 3, 1.3, 1e-3
    p = small_problem(1, n=n)
    O, aux = orc.forward(p["Q"], p["K"], p["V"], p["W"], beta, p["gate_w"], p["gate_b"],
                         p["omega"], L, eps=eps, gate_per_head=per_head, want_aux=True)
    _, f = orc.gate(p["Q"], p["gate_w"], p["gate_b"], p["omega"], L, gate_per_head=per_head)
    assert np.allclose(aux["f"], f)
    B, H = p["Q"].shape[:2]
    for b in range(B):
        for h in range(H):
            QF = filter_by_block_means(p["Q"][b, h], f[b, h])
            KF = filter_by_block_means(p["K"][b, h], f[b, h])
            want = brute_force_attention(QF, KF, p["V"][b, h], p["W"], beta, eps)
            assert np.max(np.abs(O[b, h] - want)) < 1e-12 * max(1.0, np.abs(want).max())


def test_forward_invariants():
    L, eps = 3, 1e-6
    p = small_problem(2, n=64)
    args = (p["W"], 1.0, p["gate_w"], p["gate_b"], p["omega"], L)
    O, aux = orc.forward(p["Q"], p["K"], p["V"], *args, eps=eps, want_aux=True)
    # sub-convex combination of value rows (features are non-negative)
    s = (aux["D"] - eps) / aux["D"]
    vmin, vmax = p["V"].min(axis=2, keepdims=True), p["V"].max(axis=2, keepdims=True)
    lo = np.minimum(vmin * s[..., None], vmax * s[..., None])
    hi = np.maximum(vmin * s[..., None], vmax * s[..., None])
    assert np.all(O >= lo - 1e-12) and np.all(O <= hi + 1e-12)
    # V = ones => O = (D - eps)/D
    O1, aux1 = orc.forward(p["Q"], p["K"], np.ones_like(p["V"]), *args, eps=eps, want_aux=True)
    assert np.allclose(O1, np.broadcast_to(((aux1["D"] - eps) / aux1["D"])[..., None], O1.shape),
                       atol=1e-13)
    # z and S really are the key sums: z = S applied to V = ones
    assert np.allclose(aux1["S"].sum(axis=-1) / p["V"].shape[-1], aux1["z"], atol=1e-12)
    # sampled rows agree with the full run and leave the rest untouched
    rows = np.array([0, 5, 63])
    Os = orc.forward(p["Q"], p["K"], p["V"], *args, eps=eps, sample_rows=rows)
    assert np.allclose(Os[:, :, rows], O[:, :, rows], atol=0) and np.isnan(Os[:, :, 1]).all()


def test_unit_filter_reduces_to_plain_random_feature_attention():
    # "NoWavelet" ablation (Appendix E) as a special case: f == 1 (sigmoid(0) * 2).
    L, eps = 4, 1e-4
    p = small_problem(3, n=32, gates=False)
    om = np.full(L + 1, 2.0)
    O = orc.forward(p["Q"], p["K"], p["V"], p["W"], 0.8, None, None, om, L, eps=eps)
    for b in range(2):
        for h in range(2):
            want = brute_force_attention(p["Q"][b, h], p["K"][b, h], p["V"][b, h], p["W"], 0.8, eps)
            assert np.max(np.abs(O[b, h] - want)) < 1e-12
    # joint permutation of (K, V) rows leaves O unchanged when all gates are equal
    perm = np.random.default_rng(0).permutation(32)
    Op = orc.forward(p["Q"], p["K"][:, :, perm], p["V"][:, :, perm], p["W"], 0.8, None, None, om,
                     L, eps=eps)
    assert np.allclose(Op, O, atol=1e-12)


def test_bandwidth_only_acts_through_eps():
    # ReLU is positively homogeneous: O(beta, eps) = O(c beta, eps / c^2).
    L = 3
    p = small_problem(4, n=64)
    a = orc.forward(p["Q"], p["K"], p["V"], p["W"], 1.0, p["gate_w"], p["gate_b"], p["omega"], L,
                    eps=1e-2)
    b = orc.forward(p["Q"], p["K"], p["V"], p["W"], 2.0, p["gate_w"], p["gate_b"], p["omega"], L,
                    eps=1e-2 / 4)
    assert np.max(np.abs(a - b)) < 1e-13
    c = orc.forward(p["Q"], p["K"], p["V"], p["W"], 2.0, p["gate_w"], p["gate_b"], p["omega"], L,
                    eps=1e-2)
    assert np.max(np.abs(a - c)) > 1e-6      # and it does act through eps


# ---------------------------------------------------------------- backward: finite differences
def _loss(p, dO, L, eps, per_head, beta):
    O = orc.forward(p["Q"], p["K"], p["V"], p["W"], beta, p["gate_w"], p["gate_b"], p["omega"],
                    L, eps=eps, gate_per_head=per_head)
    return float((O * dO).sum())


@pytest.mark.parametrize("n,per_head", [(64, 1), (40, 1), (64, 0)])
def test_backward_matches_central_finite_differences(n, per_head):
    L, eps, beta, h = 3, 5e-2, 0.9, 1e-6
    p = small_problem(10 + n + per_head, B=2, H=2, n=n, d=8, m=16)
    rng = np.random.default_rng(99)
    dO = rng.standard_normal(p["Q"].shape)
    g = orc.backward(p["Q"], p["K"], p["V"], p["W"], beta, p["gate_w"], p["gate_b"], p["omega"],
                     dO, L, eps=eps, gate_per_head=per_head)
    names = {"Q": "dQ", "K": "dK", "V": "dV", "gate_w": "dgate_w", "gate_b": "dgate_b",
             "omega": "domega"}
    for key, gname in names.items():
        grad = g[gname]
        flat_idx = rng.choice(p[key].size, size=min(p[key].size, 60), replace=False)
        def central(idx, step):
            q = {k: (None if v is None else v.copy()) for k, v in p.items()}
            q[key].reshape(-1)[idx] += step
            up = _loss(q, dO, L, eps, per_head, beta)
            q[key].reshape(-1)[idx] -= 2 * step
            dn = _loss(q, dO, L, eps, per_head, beta)
            return (up - dn) / (2 * step)

        scale = max(np.abs(grad).max(), 1e-30)
        fd = np.zeros(len(flat_idx))
        for j, idx in enumerate(flat_idx):
            fd[j] = central(idx, h)
            if abs(fd[j] - grad.reshape(-1)[idx]) > 2e-6 * scale + 1e-7:
                # a ReLU kink inside [x-h, x+h] spoils the difference quotient (the loss is
                # only piecewise smooth); a 100x narrower bracket almost surely avoids it.
                fd[j] = central(idx, h / 100)
        got = grad.reshape(-1)[flat_idx]
        if key == "gate_b" and not per_head:
            # only bias row 0 is used by the batch-wide gate
            assert np.all(grad[1:] == 0)
        assert np.max(np.abs(got - fd)) < 1e-5 * scale + 1e-7, (key, np.max(np.abs(got - fd)), scale)
    fd_beta = (_loss(p, dO, L, eps, per_head, beta + h) - _loss(p, dO, L, eps, per_head, beta - h)) / (2 * h)
    assert g["dbeta"] == pytest.approx(fd_beta, rel=1e-5, abs=1e-8)
    # closed form implied by homogeneity equals the generic chain-rule value
    assert g["dbeta"] == pytest.approx(g["dbeta_closed"], rel=1e-9, abs=1e-13)
    assert abs(g["dbeta"]) > 1e-4            # eps is large enough that this pin is not vacuous


def test_backward_bandwidth_floor_kills_gradient():
    L = 3
    p = small_problem(20, n=32)
    dO = np.random.default_rng(1).standard_normal(p["Q"].shape)
    g = orc.backward(p["Q"], p["K"], p["V"], p["W"], 0.1, p["gate_w"], p["gate_b"], p["omega"],
                     dO, L, eps=1e-2, bw_floor=0.5)
    assert g["dbeta"] == 0.0 and g["dbeta_closed"] == 0.0


def test_backward_dD_identity():
    # dL/dD_t = -sum_c dO[t,c] O[t,c] / D_t, so sum_t dD_t is computable from the forward
    # alone; with it the closed-form bandwidth gradient can be pinned without the backward.
    L, eps, beta = 3, 1e-2, 1.4
    p = small_problem(21, n=64)
    dO = np.random.default_rng(2).standard_normal(p["Q"].shape)
    O, aux = orc.forward(p["Q"], p["K"], p["V"], p["W"], beta, p["gate_w"], p["gate_b"],
                         p["omega"], L, eps=eps, want_aux=True)
    sum_dD = float((-(dO * O).sum(axis=-1) / aux["D"]).sum())
    g = orc.backward(p["Q"], p["K"], p["V"], p["W"], beta, p["gate_w"], p["gate_b"], p["omega"],
                     dO, L, eps=eps)
    assert g["dbeta_closed"] == pytest.approx(2 * eps / beta * sum_dD, rel=1e-12)
