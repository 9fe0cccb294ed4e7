"""Seeded synthetic inputs for the WERSA operator, shared by the tests, the smoke check and
the benchmark.  This module holds none of the method's arithmetic: it only draws random
tensors of the shapes and value distributions of the five benchmark configurations (and two
shapes with the paper's own hyper-parameters) and
rounds them to the storage type the configuration names.

Recipe (every configuration): one numpy `default_rng(seed)`; Q, K, V and (where used) dO are
drawn in that order as float64 standard normals, scaled, cast to float32 and, for bf16
configurations, rounded to nearest-even bf16.  W comes from its own seed, the gating
parameters from theirs.  The values returned are float32 arrays that are exactly
representable in the storage type, so the float64 oracle and the GPU see identical numbers;
`to_bf16_bits` gives the uint16 image a device tensor is built from.
"""
import numpy as np

# name -> shape/dtype/seeds.  "scale" multiplies Q, K, V; gates: None = initial values
# (gate_w = 0, gate_b = 0), else the standard deviation of iid normal gate_w / gate_b.
CONFIGS = {
    "cfg1_single_head_fp32": dict(B=1, H=1, n=1024, d=64, L=3, m=64, dtype="f32", scale=1.0,
                                  seed=0, w_seed=1, gate_std=None, gate_seed=None, backward=False),
    "cfg2_text_bf16": dict(B=8, H=8, n=4096, d=64, L=4, m=256, dtype="bf16", scale=0.5,
                           seed=2, w_seed=1002, gate_std=0.1, gate_seed=2002, backward=False),
    "cfg3_vision_bf16": dict(B=64, H=12, n=1024, d=64, L=5, m=128, dtype="bf16", scale=1.0,
                             seed=3, w_seed=1003, gate_std=0.1, gate_seed=2003, backward=False),
    "cfg4_long_bf16": dict(B=1, H=8, n=131072, d=64, L=8, m=256, dtype="bf16", scale=0.125,
                           seed=4, w_seed=1004, gate_std=None, gate_seed=None, backward=False),
    "cfg5_train_bf16": dict(B=4, H=8, n=16384, d=64, L=6, m=256, dtype="bf16", scale=1.0,
                            seed=5, w_seed=1005, gate_std=0.1, gate_seed=2005, backward=True),
    # Shapes with the paper's own hyper-parameters (L = 2, m = 1024; heads of 32 and 16 dimensions), for
    # `bench.py --workload`: a text-classification-sized batch and one 128k-token sequence.
    "paper_text_bf16": dict(B=32, H=4, n=4096, d=32, L=2, m=1024, dtype="bf16", scale=1.0,
                            seed=6, w_seed=1006, gate_std=0.1, gate_seed=2006, backward=True),
    "paper_long_bf16": dict(B=1, H=4, n=131072, d=16, L=2, m=1024, dtype="bf16", scale=0.25,
                            seed=7, w_seed=1007, gate_std=0.1, gate_seed=2007, backward=False),
}


def round_to_bf16(x):
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (bits + 0x7FFF + ((bits >> 16) & 1)) & 0xFFFF0000
    return rounded.astype(np.uint32).view(np.float32).reshape(np.shape(x))


def to_bf16_bits(x):
    """uint16 bf16 image of float32 values that are already exactly representable in bf16."""
    bits = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    assert not np.any(bits & 0xFFFF), "values are not bf16-representable"
    return (bits >> 16).astype(np.uint16).reshape(np.shape(x))


def make_inputs(B, H, n, d, L, m, dtype="f32", scale=1.0, seed=0, w_seed=1, gate_std=None,
                gate_seed=None, backward=False, beta=1.0, mean_shift=0.0, orthogonal_w=False, **_unused):
    """Draw one problem instance.  Returns a dict of float32 numpy arrays:
    Q, K, V (B,H,n,d), W (d,m), beta (1,), gate_w (H,d,L+1), gate_b (H,L+1), omega (L+1,),
    and dO (B,H,n,d) when backward=True.  `mean_shift` adds a constant to Q so that the
    pooled query, and with it the gate, is not ~0 (iid zero-mean inputs pool to ~0)."""
    rng = np.random.default_rng(seed)
    shape = (B, H, n, d)

    def draw():
        x = (rng.standard_normal(shape) * scale).astype(np.float32)
        return x

    Q = draw()
    if mean_shift:
        Q = (Q + np.float32(mean_shift)).astype(np.float32)
    K = draw()
    V = draw()
    out = dict(Q=Q, K=K, V=V)
    if backward:
        out["dO"] = rng.standard_normal(shape).astype(np.float32)
    W = np.random.default_rng(w_seed).standard_normal((d, m))
    if orthogonal_w:
        # the paper allows an orthogonal R in place of the Gaussian one: blocks of d orthonormal columns (QR of
        # the Gaussian draw, block by block), rescaled to the Gaussian columns' expected norm sqrt(d)
        for c0 in range(0, m, d):
            q, _ = np.linalg.qr(W[:, c0:c0 + d])
            W[:, c0:c0 + q.shape[1]] = q[:, :min(d, m - c0)] * np.sqrt(d)
    out["W"] = W.astype(np.float32)
    if gate_std is None:
        out["gate_w"] = np.zeros((H, d, L + 1), dtype=np.float32)
        out["gate_b"] = np.zeros((H, L + 1), dtype=np.float32)
    else:
        grng = np.random.default_rng(gate_seed)
        out["gate_w"] = (grng.standard_normal((H, d, L + 1)) * gate_std).astype(np.float32)
        out["gate_b"] = (grng.standard_normal((H, L + 1)) * gate_std).astype(np.float32)
    out["omega"] = np.ones(L + 1, dtype=np.float32)
    out["beta"] = np.full(1, beta, dtype=np.float32)
    if dtype == "bf16":
        for key in ("Q", "K", "V", "W", "dO"):
            if key in out:
                out[key] = round_to_bf16(out[key])
    return out


def make_config(name, **overrides):
    """Inputs of a named benchmark configuration; overrides shrink it (e.g. B=1, H=2)."""
    cfg = dict(CONFIGS[name])
    cfg.update(overrides)
    return cfg, make_inputs(**cfg)


def to_device(x, dtype, device="cuda"):
    """float32 numpy array (bf16-representable when dtype is bf16) -> torch CUDA tensor of that storage type.
    Pure data movement: the bf16 tensor is built from the 16-bit image of the values."""
    import torch
    if dtype == "bf16":
        bits = to_bf16_bits(x).view(np.int16)
        return torch.from_numpy(bits.copy()).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(device)


def device_inputs(inp, dtype, device="cuda"):
    """Device copies of one problem instance: Q, K, V, W, dO in the storage type, parameters as float32."""
    out = {}
    for key in ("Q", "K", "V", "W", "dO"):
        if key in inp:
            out[key] = to_device(inp[key], dtype, device)
    for key in ("beta", "gate_w", "gate_b", "omega"):
        out[key] = None if inp.get(key) is None else to_device(inp[key], "f32", device)
    return out
