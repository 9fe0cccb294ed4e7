"""GPU parity tests: the CUDA library, called through its C ABI (ctypes binding), against the
float64 CPU oracle on the same seeded inputs.  Tolerances: fp32 storage max normalised error
1e-4; bf16 storage max 2e-2 and mean 3e-3 (errors normalised by max(|ref|, slab rms))."""
import numpy as np
import pytest

import wersa_inputs as wi
from oracle import wersa_oracle as orc
from tests.util import device_inputs, normalised_error, small_vector_error, to_device, to_numpy64

pytestmark = pytest.mark.gpu

F32_MAX = 1e-4
BF16_MAX, BF16_MEAN = 2e-2, 3e-3


def _ctx(cfg, **kw):
    import paper_2507_08637_b200 as wersa
    args = dict(dtype=cfg["dtype"], grad_dtype="f32", eps=cfg.get("eps", 1e-6),
                gate_per_head=cfg.get("gate_per_head", 1))
    args.update(kw)
    return wersa.wersa_create(cfg["B"], cfg["H"], cfg["n"], cfg["d"], cfg["L"], cfg["m"], **args)


def _oracle_forward(cfg, inp, **kw):
    return orc.forward(inp["Q"], inp["K"], inp["V"], inp["W"], float(inp["beta"][0]), inp["gate_w"],
                       inp["gate_b"], inp["omega"], cfg["L"], eps=cfg.get("eps", 1e-6),
                       gate_per_head=cfg.get("gate_per_head", 1), **kw)


def _check(got, ref, dtype, what=""):
    err = normalised_error(got, ref)
    if dtype == "f32":
        assert err.max() <= F32_MAX, (what, err.max())
    else:
        assert err.max() <= BF16_MAX, (what, "max", err.max())
        assert err.mean() <= BF16_MEAN, (what, "mean", err.mean())
    return err


# ---------------------------------------------------------------- Haar filter kernel
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("n,L", [(8, 3), (256, 8), (1024, 5), (2048, 8), (1000, 3), (300, 4), (77, 2)])
def test_haar_filter_kernel(n, L, dtype):
    import torch
    B, H, d = 2, 3, 64
    rng = np.random.default_rng(n * 10 + L)
    X = (rng.standard_normal((B, H, n, d)) + 0.5).astype(np.float32)
    # multi-scale structure so that every band carries energy
    X += np.sin(np.arange(n)[None, None, :, None] * 2 * np.pi / 64.0).astype(np.float32)
    if dtype == "bf16":
        X = wi.round_to_bf16(X)
    f = rng.uniform(0.2, 1.5, (B, H, L + 1)).astype(np.float32)
    cfg = dict(B=B, H=H, n=n, d=d, L=L, m=64, dtype=dtype)
    ctx = _ctx(cfg)
    got = ctx.haar_filter(to_device(X, dtype), torch.from_numpy(f).cuda())
    torch.cuda.synchronize()
    got = to_numpy64(got)
    for b in range(B):
        for h in range(H):
            ref = orc.haar_filter(X[b, h].astype(np.float64), f[b, h].astype(np.float64))
            scale = np.abs(ref).max()
            tol = 2e-6 if dtype == "f32" else 2.0 ** -8
            assert np.max(np.abs(got[b, h] - ref)) <= tol * scale, (b, h)


# ---------------------------------------------------------------- gate
@pytest.mark.parametrize("per_head", [1, 0])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gate_and_saved_tensors(dtype, per_head):
    cfg = dict(B=2, H=3, n=1280, d=64, L=4, m=64, dtype=dtype, gate_per_head=per_head)
    inp = wi.make_inputs(**cfg, seed=11, w_seed=12, gate_std=0.3, gate_seed=13, mean_shift=0.4)
    ctx = _ctx(cfg)
    dev = device_inputs(inp, dtype)
    ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    qbar, f = orc.gate(inp["Q"], inp["gate_w"], inp["gate_b"], inp["omega"], cfg["L"], gate_per_head=per_head)
    assert np.max(np.abs(to_numpy64(ctx.saved("qbar")) - qbar)) < 2e-6
    assert np.max(np.abs(to_numpy64(ctx.saved("f")) - f)) < 2e-6
    # the gate must actually have moved away from sigmoid(0)
    assert np.abs(f - 0.5).max() > 0.05


# ---------------------------------------------------------------- forward, small shapes
SMALL = [
    dict(B=1, H=1, n=8, d=64, L=3, m=64),
    dict(B=2, H=2, n=64, d=64, L=3, m=128),
    dict(B=1, H=3, n=1024, d=64, L=5, m=256),
    dict(B=2, H=1, n=1000, d=64, L=3, m=64),      # ragged: not a multiple of 32 nor of 2^L
    dict(B=1, H=2, n=4100, d=64, L=8, m=128),     # several Haar tiles and a ragged tail
    dict(B=3, H=2, n=512, d=64, L=8, m=256, gate_per_head=0),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", range(len(SMALL)))
def test_forward_small_simt(case, dtype):
    import paper_2507_08637_b200 as wersa
    import torch
    cfg = dict(SMALL[case], dtype=dtype)
    inp = wi.make_inputs(**cfg, seed=100 + case, w_seed=200 + case, gate_std=0.3, gate_seed=300 + case,
                         mean_shift=0.25, scale=0.7)
    ctx = _ctx(cfg, flags=wersa.WERSA_FLAG_SIMT_ONLY)
    dev = device_inputs(inp, dtype)
    O = ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                    dev["omega"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    ref, aux = _oracle_forward(cfg, inp, want_aux=True)
    _check(to_numpy64(O), ref, dtype, "O")
    # key summary and normaliser (library keeps them without the 1/(bw sqrt(m)) factor)
    c = 1.0 / (max(float(inp["beta"][0]), 1e-6) * np.sqrt(cfg["m"]))
    errS = normalised_error(to_numpy64(ctx.saved("S")) * c, aux["S"])
    errz = normalised_error(to_numpy64(ctx.saved("z")) * c, aux["z"])
    assert errS.max() < 1e-4 and errz.max() < 1e-4
    assert ctx.launch_count(0) >= 5


TC_SMALL = [
    dict(B=1, H=1, n=128, d=64, L=3, m=128),      # one tile, one unit
    dict(B=1, H=1, n=128, d=64, L=7, m=256),      # one tile, two feature halves
    dict(B=1, H=2, n=384, d=64, L=5, m=256),      # odd number of tiles
    dict(B=2, H=2, n=1152, d=64, L=4, m=128),     # more tiles than ring stages, alternating warpgroups
    dict(B=1, H=1, n=2560, d=64, L=8, m=256),     # 20 tiles in one CTA chunk set
    dict(B=2, H=3, n=4096, d=64, L=8, m=256, gate_per_head=0),
    dict(B=2, H=1, n=1000, d=64, L=3, m=128),     # ragged: last block is partly past the end
    dict(B=1, H=2, n=4100, d=64, L=8, m=256),     # ragged tail of 4 rows in a 256-row Haar block
    dict(B=1, H=1, n=77, d=64, L=2, m=128),       # shorter than one tile
    dict(B=10, H=8, n=1024, d=64, L=6, m=256),    # 80 slabs: one chunk of four blocks per slab, no reduction launch
]


@pytest.mark.parametrize("case", range(len(TC_SMALL)))
def test_forward_small_tensor_core(case):
    import torch
    cfg = dict(TC_SMALL[case], dtype="bf16")
    inp = wi.make_inputs(**cfg, seed=700 + case, w_seed=800 + case, gate_std=0.3, gate_seed=900 + case,
                         mean_shift=0.25, scale=0.7)
    ctx = _ctx(cfg)
    assert ctx.uses_tensor_cores()
    dev = device_inputs(inp, "bf16")
    O = ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                    dev["omega"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    ref, aux = _oracle_forward(cfg, inp, want_aux=True)
    c = 1.0 / (max(float(inp["beta"][0]), 1e-6) * np.sqrt(cfg["m"]))
    errS = normalised_error(to_numpy64(ctx.saved("S")) * c, aux["S"])
    errz = normalised_error(to_numpy64(ctx.saved("z")) * c, aux["z"])
    assert errS.max() < 2e-2 and errz.max() < 5e-3, (errS.max(), errz.max())
    _check(to_numpy64(O), ref, "bf16", "O")


# ---------------------------------------------------------------- head dimensions below 64, more than 256 features
NARROW = [
    dict(B=2, H=2, n=640, d=32, L=2, m=128),       # the paper's head dimension of its text models (Sec. 4.1)
    dict(B=1, H=3, n=1000, d=16, L=3, m=256),      # Sec. 4.5: 64 dimensions over 4 heads; ragged n
    dict(B=2, H=1, n=300, d=32, L=4, m=64, gate_per_head=0),
    dict(B=1, H=2, n=2304, d=8, L=8, m=256),
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", range(len(NARROW)))
def test_forward_and_backward_with_narrow_heads(case, dtype):
    """head_dim < 64 (run as the zero-padded 64-wide problem) against the oracle on the narrow tensors
    themselves: the output, the saved q-bar, S', z' and every gradient."""
    import torch
    cfg = dict(NARROW[case], dtype=dtype, eps=1e-3)
    inp = wi.make_inputs(**cfg, seed=1400 + case, w_seed=1500 + case, gate_std=0.3, gate_seed=1600 + case,
                         mean_shift=0.25, scale=0.7, backward=True)
    ctx = _ctx(cfg)
    assert ctx.uses_tensor_cores() == (dtype == "bf16" and cfg["m"] >= 128)
    dev = device_inputs(inp, dtype)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    O = ctx.forward(*args)
    torch.cuda.synchronize()
    assert ctx.query_status() == 0 and tuple(O.shape) == inp["Q"].shape
    ref, aux = _oracle_forward(cfg, inp, want_aux=True)
    _check(to_numpy64(O), ref, dtype, "O")
    tol = 1e-4 if not ctx.uses_tensor_cores() else 2e-2
    c = 1.0 / (max(float(inp["beta"][0]), 1e-6) * np.sqrt(cfg["m"]))
    S = to_numpy64(ctx.saved("S"))
    assert S.shape[-1] == cfg["d"]
    assert normalised_error(S * c, aux["S"]).max() < tol
    assert normalised_error(to_numpy64(ctx.saved("z")) * c, aux["z"]).max() < tol
    assert to_numpy64(ctx.saved("qbar")).shape[-1] == cfg["d"]
    grads = ctx.backward(*args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    assert tuple(grads["dQ"].shape) == inp["Q"].shape and tuple(grads["dgate_w"].shape) == inp["gate_w"].shape
    _check_backward(cfg, inp, grads)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_narrow_heads_equal_the_padded_problem(dtype):
    """The narrow problem and the same tensors zero-padded to 64 columns by the caller agree: bit for bit on
    the fp32 path (which pads them itself), to bf16 rounding on the tensor-core path (whose tensor maps
    zero-fill the narrow tensors; only the order of the mean-pool sums differs)."""
    import torch
    cfg = dict(B=2, H=2, n=900, d=32, L=3, m=256, dtype=dtype)
    inp = wi.make_inputs(**cfg, seed=1450, w_seed=1451, gate_std=0.3, gate_seed=1452, mean_shift=0.25, scale=0.7)
    dev = device_inputs(inp, dtype)
    O = _ctx(cfg).forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                          dev["omega"])
    Qp, Kp, Vp = (torch.nn.functional.pad(dev[k], (0, 32)).contiguous() for k in ("Q", "K", "V"))
    Wp = torch.cat([dev["W"], torch.zeros_like(dev["W"])], dim=0).contiguous()
    gwp = torch.cat([dev["gate_w"], torch.zeros_like(dev["gate_w"])], dim=1).contiguous()
    O64 = _ctx(dict(cfg, d=64)).forward(Qp, Kp, Vp, Wp, dev["beta"], gwp, dev["gate_b"], dev["omega"])
    torch.cuda.synchronize()
    assert float(O64[..., 32:].abs().max()) == 0.0
    if dtype == "f32":
        assert torch.equal(O64[..., :32].contiguous(), O)
    else:
        diff = (O64[..., :32].float() - O.float()).abs().max()
        assert float(diff) <= 2.0 ** -7 * float(O.float().abs().max())


WIDE = [
    dict(B=1, H=2, n=1024, d=64, L=2, m=1024),       # Sec. 3.3: L = 2, m = 1024
    dict(B=2, H=1, n=3000, d=64, L=5, m=512),        # several chunks per slab (reduction launch per group), ragged
    dict(B=1, H=1, n=40000, d=64, L=8, m=768),       # many chunks, three groups
    dict(B=12, H=16, n=512, d=64, L=4, m=512),       # 192 slabs: several work items per CTA, one chunk per slab
    dict(B=2, H=4, n=700, d=32, L=2, m=1024, gate_per_head=0),   # the paper's text-model shape: d = 32, m = 1024
]


@pytest.mark.parametrize("case", range(len(WIDE)))
def test_forward_with_wide_feature_maps(case):
    """m = 512, 768, 1024 (groups of 256 features combined by their denominators) against the oracle on the
    whole feature map: the output and the saved S', z'; twice, bit-identical."""
    import torch
    cfg = dict(WIDE[case], dtype="bf16")
    inp = wi.make_inputs(**cfg, seed=1700 + case, w_seed=1800 + case, gate_std=0.3, gate_seed=1900 + case,
                         mean_shift=0.25, scale=0.7)
    ctx = _ctx(cfg)
    assert ctx.uses_tensor_cores()
    dev = device_inputs(inp, "bf16")
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    O = ctx.forward(*args).clone()
    O2 = ctx.forward(*args)
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    assert torch.equal(O.view(torch.int16), O2.view(torch.int16))
    ref, aux = _oracle_forward(cfg, inp, want_aux=True)
    c = 1.0 / (max(float(inp["beta"][0]), 1e-6) * np.sqrt(cfg["m"]))
    errS = normalised_error(to_numpy64(ctx.saved("S")) * c, aux["S"])
    errz = normalised_error(to_numpy64(ctx.saved("z")) * c, aux["z"])
    assert errS.max() < 2e-2 and errz.max() < 5e-3, (errS.max(), errz.max())
    _check(to_numpy64(O), ref, "bf16", "O")


WIDE_BWD = [
    dict(B=1, H=2, n=1024, d=64, L=2, m=1024),
    dict(B=2, H=1, n=1500, d=64, L=5, m=512),
    dict(B=2, H=2, n=700, d=32, L=2, m=1024, gate_per_head=0),
    dict(B=1, H=3, n=2304, d=64, L=6, m=768),
]


@pytest.mark.parametrize("grad_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", range(len(WIDE_BWD)))
def test_backward_with_wide_feature_maps(case, grad_dtype):
    """Gradients with m = 512, 768, 1024: every group runs the tensor-core backward kernels with the whole map's
    denominator and dD', and dQ_F, dV, dK_F accumulate over the groups."""
    import torch
    if grad_dtype == "bf16" and case not in (0, 2):
        pytest.skip("bf16 gradients: two cases")
    cfg = dict(WIDE_BWD[case], dtype="bf16", eps=1e-3)
    inp = wi.make_inputs(**cfg, seed=2100 + case, w_seed=2200 + case, gate_std=0.3, gate_seed=2300 + case,
                         mean_shift=0.25, scale=0.7, backward=True)
    ctx = _ctx(cfg, grad_dtype=grad_dtype)
    assert ctx.uses_tensor_cores()
    dev = device_inputs(inp, "bf16")
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    ctx.forward(*args)
    grads = ctx.backward(*args, dev["dO"])
    grads2 = ctx.backward(*args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    for k in ("dQ", "dK", "dV"):
        assert torch.equal(grads[k], grads2[k]), k   # accumulation in launch order: the same bits every time
    _check_backward(cfg, inp, grads)


# ---------------------------------------------------------------- sequence shards (one GPU standing in for several)
SHARDED = [
    (dict(B=2, H=2, n=3000, d=64, L=5, m=256), [1024, 1024, 952]),
    (dict(B=1, H=3, n=2304, d=32, L=8, m=128, gate_per_head=0), [1536, 768]),
    (dict(B=1, H=1, n=70000, d=64, L=6, m=256), [32768, 37232]),       # several chunks per shard
]


@pytest.mark.parametrize("case", range(len(SHARDED)))
def test_sequence_sharded_forward(case):
    """The four shard steps on contexts of the shards' lengths, with the two sums between them taken here (on
    several GPUs they are all-reduces): the shards' outputs put together meet the oracle's forward on the whole
    sequence, and the whole-sequence context's forward to bf16 rounding."""
    import torch
    cfg, lens = SHARDED[case]
    cfg = dict(cfg, dtype="bf16")
    assert sum(lens) == cfg["n"] and all(l % (1 << cfg["L"]) == 0 for l in lens[:-1])
    inp = wi.make_inputs(**cfg, seed=2500 + case, w_seed=2600 + case, gate_std=0.3, gate_seed=2700 + case,
                         mean_shift=0.25, scale=0.7)
    dev = device_inputs(inp, "bf16")
    starts = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    shards = [{k: dev[k][:, :, a:b].contiguous() for k in ("Q", "K", "V")} for a, b in zip(starts[:-1], starts[1:])]
    ctxs = [_ctx(dict(cfg, n=l)) for l in lens]
    qsum = sum(c.shard_pool(s["Q"], dev["W"]) for c, s in zip(ctxs, shards))
    S_total = z_total = None
    for c, s in zip(ctxs, shards):
        c.shard_gate(qsum, cfg["n"], dev["gate_w"], dev["gate_b"], dev["omega"])
        S, z = c.shard_keys(s["K"], s["V"])
        S_total = S.clone() if S_total is None else S_total + S
        z_total = z.clone() if z_total is None else z_total + z
    O = torch.cat([c.shard_output(s["Q"], S_total, z_total, dev["beta"]) for c, s in zip(ctxs, shards)], dim=2)
    torch.cuda.synchronize()
    assert all(c.query_status() == 0 for c in ctxs)
    ref, aux = _oracle_forward(cfg, inp, want_aux=True)
    _check(to_numpy64(O), ref, "bf16", "O")
    f = to_numpy64(ctxs[0].saved("f"))
    assert np.max(np.abs(f - aux["f"])) < 2e-6
    whole = _ctx(cfg).forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                              dev["omega"])
    torch.cuda.synchronize()
    diff = (whole.float() - O.float()).abs().max()
    assert float(diff) <= 2.0 ** -6 * float(whole.float().abs().max())


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_forward_with_orthogonal_projection(dtype):
    """The projection matrix is an input: an orthogonal R (Sec. 3.1, step 7 allows orthogonal or Gaussian),
    drawn as orthonormal blocks of d columns, goes through the same kernels."""
    import torch
    cfg = dict(B=2, H=2, n=1500, d=64, L=4, m=256, dtype=dtype)
    inp = wi.make_inputs(**cfg, seed=2800, w_seed=2801, gate_std=0.3, gate_seed=2802, mean_shift=0.25, scale=0.7,
                         orthogonal_w=True)
    W = inp["W"].astype(np.float64)
    assert np.allclose(W[:, :64].T @ W[:, :64], 64.0 * np.eye(64), atol=1e-3 if dtype == "f32" else 0.5)   # (bf16: rounded entries)
    ctx = _ctx(cfg)
    dev = device_inputs(inp, dtype)
    O = ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _check(to_numpy64(O), _oracle_forward(cfg, inp), dtype, "O")


SHARDED_BWD = [
    (dict(B=2, H=2, n=2000, d=64, L=5, m=256), [1024, 976]),
    (dict(B=1, H=3, n=1536, d=64, L=8, m=128, gate_per_head=0), [768, 512, 256]),
]


@pytest.mark.parametrize("case", range(len(SHARDED_BWD)))
def test_sequence_sharded_backward(case):
    """Forward and backward shard steps on contexts of the shards' lengths, every sum between them taken here
    (all-reduces on several GPUs): the shards' dQ, dK, dV put together and the parameter gradients meet the
    oracle's backward on the whole sequence."""
    import torch
    cfg, lens = SHARDED_BWD[case]
    cfg = dict(cfg, dtype="bf16", eps=1e-3)
    assert sum(lens) == cfg["n"] and all(l % (1 << cfg["L"]) == 0 for l in lens[:-1])
    inp = wi.make_inputs(**cfg, seed=2900 + case, w_seed=3000 + case, gate_std=0.3, gate_seed=3100 + case,
                         mean_shift=0.25, scale=0.7, backward=True)
    dev = device_inputs(inp, "bf16")
    starts = np.concatenate([[0], np.cumsum(lens)]).astype(int)
    shards = [{k: dev[k][:, :, a:b].contiguous() for k in ("Q", "K", "V", "dO")} for a, b in zip(starts[:-1], starts[1:])]
    ctxs = [_ctx(dict(cfg, n=l)) for l in lens]
    pairs = list(zip(ctxs, shards))
    qsum = sum(c.shard_pool(s["Q"], dev["W"]) for c, s in pairs)
    Ss, zs = [], []
    for c, s in pairs:
        c.shard_gate(qsum, cfg["n"], dev["gate_w"], dev["gate_b"], dev["omega"])
        S, z = c.shard_keys(s["K"], s["V"])
        Ss.append(S.clone()); zs.append(z.clone())
    S_total, z_total = sum(Ss), sum(zs)
    for c, s in pairs:
        c.shard_output(s["Q"], S_total, z_total, dev["beta"])
    parts = [c.shard_backward_queries(s["Q"], dev["beta"], s["dO"]) for c, s in pairs]
    dS_total = sum(p[0].clone() for p in parts)
    dz_total = sum(p[1].clone() for p in parts)
    kv = [c.shard_backward_keys(s["K"], s["V"], dS_total, dz_total) for c, s in pairs]
    df_total = sum(r[2].clone() for r in kv)
    sumdD_total = sum(r[3].clone() for r in kv)
    gates = [c.shard_backward_gate(s["Q"], df_total, sumdD_total, cfg["n"], dev["beta"], dev["gate_w"], dev["omega"])
             for c, s in pairs]
    torch.cuda.synchronize()
    assert all(c.query_status() == 0 for c in ctxs)
    grads = dict(gates[0])
    grads["dQ"] = torch.cat([g["dQ"] for g in gates], dim=2)
    grads["dK"] = torch.cat([r[0] for r in kv], dim=2)
    grads["dV"] = torch.cat([r[1] for r in kv], dim=2)
    for g in gates[1:]:   # the parameter gradients are the same on every shard
        for k in ("dbeta", "dgate_w", "dgate_b", "domega"):
            assert torch.equal(g[k], gates[0][k]), k
    _check_backward(cfg, inp, grads)


def test_sharded_helpers_with_a_single_rank():
    """paper_2507_08637_b200.sharded.forward_sharded / backward_sharded without a process group (one rank holds
    the whole sequence, the all-reduces are no-ops): the same results as the oracle on that sequence."""
    import torch
    from paper_2507_08637_b200.sharded import backward_sharded, forward_sharded
    cfg = dict(B=2, H=2, n=1300, d=64, L=4, m=256, dtype="bf16", eps=1e-3)
    inp = wi.make_inputs(**cfg, seed=3200, w_seed=3201, gate_std=0.3, gate_seed=3202, mean_shift=0.25, scale=0.7,
                         backward=True)
    dev = device_inputs(inp, "bf16")
    ctx = _ctx(cfg)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    O = forward_sharded(ctx, *args)
    grads = backward_sharded(ctx, *args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _check(to_numpy64(O), _oracle_forward(cfg, inp), "bf16", "O")
    _check_backward(cfg, inp, grads)


def test_forward_is_bit_identical_run_to_run():
    import paper_2507_08637_b200 as wersa
    import torch
    cfg = dict(B=2, H=2, n=4096, d=64, L=6, m=256, dtype="bf16")
    inp = wi.make_inputs(**cfg, seed=5, w_seed=6, gate_std=0.1, gate_seed=7)
    dev = device_inputs(inp, "bf16")
    for flags in (wersa.WERSA_FLAG_SIMT_ONLY, 0):
        ctx = _ctx(cfg, flags=flags)
        a = ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                        dev["omega"]).clone()
        b = ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                        dev["omega"])
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))


@pytest.mark.parametrize("dtype,d", [("bf16", 64), ("f32", 64), ("bf16", 32)])
def test_forward_host_matches_device_forward_and_oracle(dtype, d):
    """The end-to-end entry point (host tensors in, host tensor out) gives the device-resident forward's
    bits, page-locked or pageable, and meets the oracle at the same tolerance."""
    import torch
    cfg = dict(B=2, H=3, n=1500, d=d, L=5, m=128, dtype=dtype)
    inp = wi.make_inputs(**cfg, seed=41, w_seed=42, gate_std=0.2, gate_seed=43, mean_shift=0.2)
    ctx = _ctx(cfg)
    dev = device_inputs(inp, dtype)
    params = (dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    O = ctx.forward(dev["Q"], dev["K"], dev["V"], *params).clone()
    torch.cuda.synchronize()
    for pinned in (True, False):
        host = [dev[k].cpu() for k in ("Q", "K", "V")]
        hO = torch.zeros_like(host[0])
        if pinned:
            host = [t.pin_memory() for t in host]
            hO = hO.pin_memory()
        stage = [torch.zeros_like(dev["Q"]) for _ in range(4)]
        out = ctx.forward_host(*host, *stage[:3], *params, stage[3], hO)
        torch.cuda.synchronize()
        assert ctx.query_status() == 0
        assert out is hO and torch.equal(hO, O.cpu())
        assert torch.equal(stage[0], dev["Q"]) and torch.equal(stage[3], O)
    _check(to_numpy64(hO), _oracle_forward(cfg, inp), dtype, "O")
    import paper_2507_08637_b200 as wersa
    with pytest.raises(ValueError):
        ctx.forward_host(dev["Q"], *host[1:], *stage[:3], *params, stage[3], hO)   # device tensor as host input
    with pytest.raises(wersa.WersaError) as e:
        big = torch.zeros(dev["Q"].numel() + 1, device="cuda", dtype=dev["Q"].dtype)
        ctx.forward_host(*host, big[1:].view_as(dev["Q"]), *stage[1:3], *params, stage[3], hO)
    assert e.value.status == 1


# ---------------------------------------------------------------- the five configurations
def _run_config(name, flags=0, **overrides):
    import torch
    cfg, inp = wi.make_config(name, **overrides)
    ctx = _ctx(cfg, flags=flags)
    dev = device_inputs(inp, cfg["dtype"])
    O = ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"],
                    dev["omega"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    return cfg, inp, dev, ctx, O


def test_config1_single_head_fp32():
    cfg, inp, dev, ctx, O = _run_config("cfg1_single_head_fp32")
    ref = _oracle_forward(cfg, inp)
    err = _check(to_numpy64(O), ref, "f32", "cfg1")
    # initial gate values: f = 0.5 everywhere
    assert np.allclose(to_numpy64(ctx.saved("f")), 0.5, atol=1e-7)
    print("cfg1 max err", err.max())


_ORACLE_CACHE = {}


def _oracle_forward_cached(name, cfg, inp):
    """Full-tensor oracle forward of a named configuration, computed once per test session (both arithmetic
    paths of the library are compared with the same reference)."""
    if name not in _ORACLE_CACHE:
        _ORACLE_CACHE[name] = _oracle_forward(cfg, inp, want_aux=True)
    return _ORACLE_CACHE[name]


def _check_config_forward(name, flags):
    """Every element of O, of every slab, against the oracle; the key summary and the normaliser too."""
    cfg, inp, dev, ctx, O = _run_config(name, flags=flags)
    ref, aux = _oracle_forward_cached(name, cfg, inp)
    err = _check(to_numpy64(O), ref, cfg["dtype"], name)
    c = 1.0 / (max(float(inp["beta"][0]), 1e-6) * np.sqrt(cfg["m"]))
    errS = normalised_error(to_numpy64(ctx.saved("S")).reshape(aux["S"].shape) * c, aux["S"])
    errz = normalised_error(to_numpy64(ctx.saved("z")).reshape(aux["z"].shape) * c, aux["z"])
    tolS = 2e-2 if not flags else 1e-4
    assert errS.max() <= tolS and errz.max() <= (5e-3 if not flags else 1e-4), (errS.max(), errz.max())
    # the stated bound also holds as a plain relative error wherever the reference is not small
    big = np.abs(ref) > np.sqrt(np.mean(ref ** 2, axis=(2, 3), keepdims=True))
    rel = np.abs(to_numpy64(O) - ref)[big] / np.abs(ref)[big]
    assert rel.max() <= BF16_MAX, rel.max()
    print(f"{name} flags={flags}: max {err.max():.3e} mean {err.mean():.3e} rel(|ref|>rms) {rel.max():.3e} "
          f"S {errS.max():.3e} z {errz.max():.3e}")
    return cfg, inp, dev, ctx, O


@pytest.mark.parametrize("flags", [0, 1])
def test_config2_text_bf16(flags):
    _check_config_forward("cfg2_text_bf16", flags)


@pytest.mark.parametrize("flags", [0, 1])
def test_config3_vision_bf16(flags):
    _check_config_forward("cfg3_vision_bf16", flags)


@pytest.mark.parametrize("flags", [0, 1])
def test_config4_long_sequence_bf16(flags):
    _check_config_forward("cfg4_long_bf16", flags)


def _dbeta_error(cfg, inp, got, ref_closed):
    """Error of the bandwidth gradient, normalised like every other error here: by max(|ref|, natural scale).
    dbeta = c sum_t dD_t with c = 2 eps / bw is a sum of signed terms that largely cancel (sum |dD_t| is
    3.4e3 times |sum dD_t| on the training configuration), so a per-term relative error delta moves the sum by
    about delta * sqrt(sum dD_t^2), whatever the size the sum happens to have.  That root-sum-square of the
    terms, from the oracle's own O and D (dD_t = -sum_c dO[t,c] O[t,c] / D[t]), is the scale; the error is
    |got - ref| / max(|ref|, c * sqrt(sum dD_t^2))."""
    O, aux = _oracle_forward(cfg, inp, want_aux=True)
    dD = -(np.asarray(inp["dO"], dtype=np.float64) * O).sum(-1) / aux["D"]
    bw = max(float(inp["beta"][0]), 1e-6)
    scale = 2.0 * cfg.get("eps", 1e-6) / bw * np.sqrt((dD ** 2).sum())
    return abs(got - ref_closed) / max(abs(ref_closed), scale, 1e-300)


AMBIGUOUS_MARGIN = 1e-6


def _ambiguous_rows(cfg, inp, key):
    """Rows of Q (key="Q") or K whose ReLU decision is not unique in working precision: the gradient of
    ReLU, 1[a > 0], is a 0/1 decision on a = x_F . w, and the kernels take it in fp32 while the oracle takes it
    in fp64.  Where |a| is below fp32 resolution (|a| <= 1e-6 |x_F| |w| for some feature; a dot product of 64
    terms carries about 64 * 2^-24 = 4e-6 of relative rounding) either answer is a correct one and the row's
    gradient differs by that feature's whole rank-one term.  Returns a boolean (B, H, n) mask of such rows,
    from the oracle's own filter and a float64 matmul."""
    qbar, f = orc.gate(inp["Q"], inp["gate_w"], inp["gate_b"], inp["omega"], cfg["L"],
                       gate_per_head=cfg.get("gate_per_head", 1))
    W = np.asarray(inp["W"], dtype=np.float64)
    wn = np.linalg.norm(W, axis=0)
    X = inp[key]
    out = np.zeros(X.shape[:3], dtype=bool)
    for b in range(X.shape[0]):
        for h in range(X.shape[1]):
            XF = orc.haar_filter(X[b, h].astype(np.float64), f[b, h])
            A = np.abs(XF @ W)
            scale = np.linalg.norm(XF, axis=1)[:, None] * wn[None, :]
            out[b, h] = (A <= AMBIGUOUS_MARGIN * scale).any(axis=1)
    return out


def _wavelet_block_mates(rows, block):
    """Rows (last axis) that share an aligned block of `block` rows with a marked row."""
    n = rows.shape[-1]
    pad = (-n) % block
    padded = np.concatenate([rows, np.zeros(rows.shape[:-1] + (pad,), dtype=bool)], axis=-1)
    blocks = padded.reshape(rows.shape[:-1] + (-1, block)).any(axis=-1, keepdims=True)
    return np.broadcast_to(blocks, padded.shape[:-1] + (padded.shape[-1] // block, block)).reshape(padded.shape)[..., :n]


def _check_grad(got, ref, dtype, what, ambiguous=None, levels=0):
    """Element-by-element check of dQ / dK / dV.  Rows whose ReLU decision is ambiguous (see _ambiguous_rows)
    are compared at a validity bound instead of the tolerance: one flipped feature moves the row of dX_F by a
    rank-one term, well below the row's own size.  dX = T_f(dX_F) spreads that term over the row's wavelet
    block with the weights of the block means, 1/2 for the level-1 partner, 1/4 within the level-2 block, ...:
    the rows that share a block of up to 16 rows (levels 1-4) with an ambiguous row are compared at the same
    validity bound; beyond that the share (<= 1/32 of a term that is itself a fraction of the rms) is below
    the tolerance."""
    err = normalised_error(got, ref)
    if ambiguous is not None and ambiguous.any():
        assert ambiguous.mean() <= 0.02, (what, "too many ambiguous rows", ambiguous.mean())
        near = _wavelet_block_mates(ambiguous, 1 << min(levels, 4))
        assert err[near].max() <= 1.0, (what, "ambiguous rows", err[near].max())
        err = err[~near]
    if dtype == "f32":
        assert err.max() <= F32_MAX, (what, err.max())
    else:
        assert err.max() <= BF16_MAX, (what, "max", err.max())
        assert err.mean() <= BF16_MEAN, (what, "mean", err.mean())
    return err


def _check_backward(cfg, inp, grads, sub_slabs=None):
    ref = orc.backward(inp["Q"], inp["K"], inp["V"], inp["W"], float(inp["beta"][0]), inp["gate_w"],
                       inp["gate_b"], inp["omega"], inp["dO"], cfg["L"], eps=cfg.get("eps", 1e-6),
                       gate_per_head=cfg.get("gate_per_head", 1))
    dtype = cfg["dtype"]
    _check_grad(to_numpy64(grads["dQ"]), ref["dQ"], dtype, "dQ", _ambiguous_rows(cfg, inp, "Q"), cfg["L"])
    _check_grad(to_numpy64(grads["dK"]), ref["dK"], dtype, "dK", _ambiguous_rows(cfg, inp, "K"), cfg["L"])
    _check_grad(to_numpy64(grads["dV"]), ref["dV"], dtype, "dV")
    tol = 1e-4 if dtype == "f32" else 2e-2
    for key in ("dgate_w", "dgate_b", "domega"):
        err = small_vector_error(to_numpy64(grads[key]), ref[key])
        assert err.max() <= tol, (key, err.max())
    db = float(grads["dbeta"].cpu()[0])
    rel = abs(db - ref["dbeta_closed"]) / max(abs(ref["dbeta_closed"]), 1e-300)
    err = _dbeta_error(cfg, inp, db, ref["dbeta_closed"])
    print(f"dbeta {db:.6e} ref {ref['dbeta_closed']:.6e} plain rel {rel:.3e} normalised {err:.3e}")
    assert err <= tol, (db, ref["dbeta_closed"], err)
    return ref


BWD_SMALL = [
    dict(B=1, H=1, n=64, d=64, L=3, m=64),
    dict(B=2, H=2, n=1024, d=64, L=5, m=128),
    dict(B=1, H=2, n=1000, d=64, L=8, m=256),
    dict(B=2, H=3, n=512, d=64, L=4, m=64, gate_per_head=0),
    dict(B=5, H=1, n=300, d=64, L=4, m=128),   # more batch elements than the four-way split of the domega sum, ragged n
]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("case", range(len(BWD_SMALL)))
def test_backward_small(case, dtype):
    import torch
    cfg = dict(BWD_SMALL[case], dtype=dtype, eps=1e-3)
    inp = wi.make_inputs(**cfg, seed=400 + case, w_seed=500 + case, gate_std=0.3, gate_seed=600 + case,
                         mean_shift=0.25, scale=0.7, backward=True)
    ctx = _ctx(cfg)
    dev = device_inputs(inp, dtype)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    ctx.forward(*args)
    grads = ctx.backward(*args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _check_backward(cfg, inp, grads)


@pytest.mark.parametrize("case", [1, 2, 4])
@pytest.mark.parametrize("simt", [False, True])
def test_backward_bf16_gradients(case, simt):
    """grad_dtype = bf16: dQ, dK, dV are the fp32-gradient run rounded to bf16 on the way out (the same
    arithmetic, another store), and meet the oracle at the bf16 tolerance."""
    import paper_2507_08637_b200 as wersa
    import torch
    cfg = dict(BWD_SMALL[case], dtype="bf16", eps=1e-3)
    inp = wi.make_inputs(**cfg, seed=450 + case, w_seed=550 + case, gate_std=0.3, gate_seed=650 + case,
                         mean_shift=0.25, scale=0.7, backward=True)
    dev = device_inputs(inp, "bf16")
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    flags = wersa.WERSA_FLAG_SIMT_ONLY if simt else 0
    out = {}
    for gd in ("f32", "bf16"):
        ctx = _ctx(cfg, grad_dtype=gd, flags=flags)
        assert ctx.uses_tensor_cores() == (not simt)
        ctx.forward(*args)
        out[gd] = ctx.backward(*args, dev["dO"])
        torch.cuda.synchronize()
        assert ctx.query_status() == 0
    for key in ("dQ", "dK", "dV"):
        assert out["bf16"][key].dtype == torch.bfloat16
        err = normalised_error(to_numpy64(out["bf16"][key]), to_numpy64(out["f32"][key]))
        assert err.max() <= 2.0 ** -7, (key, err.max())   # dQ is rounded twice (filter, then the mean-pool term)
    if not simt:   # dV goes from the fp32 accumulator to its store in one rounding
        assert torch.equal(out["bf16"]["dV"], out["f32"]["dV"].to(torch.bfloat16))
    for key in ("dbeta", "dgate_w", "dgate_b", "domega"):
        assert torch.equal(out["bf16"][key], out["f32"][key]), key
    # Against the oracle: the fp32-stored gradients meet the bf16 tolerance as they are; the bf16-stored ones
    # get the storage roundings on top (one for dK and dV, two for dQ; 2^-9 of the value each).
    ref = _check_backward(cfg, inp, out["f32"])
    for key in ("dQ", "dK", "dV"):
        err = normalised_error(to_numpy64(out["bf16"][key]), ref[key])
        assert err.max() <= BF16_MAX + 2.0 ** -8, (key, "max", err.max())
        assert err.mean() <= BF16_MEAN + 2.0 ** -10, (key, "mean", err.mean())


@pytest.mark.parametrize("flags", [0, 1])
def test_config5_training_step_bf16(flags):
    """The whole training configuration, every slab: O, dQ, dK, dV element by element, and the parameter
    gradients (sums over all 32 slabs) of the same run, against the oracle."""
    import torch
    name = "cfg5_train_bf16"
    cfg, inp, dev, ctx, O = _check_config_forward(name, flags)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    grads = ctx.backward(*args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    if name + "/bwd" not in _ORACLE_CACHE:
        _ORACLE_CACHE[name + "/bwd"] = orc.backward(
            inp["Q"], inp["K"], inp["V"], inp["W"], float(inp["beta"][0]), inp["gate_w"], inp["gate_b"],
            inp["omega"], inp["dO"], cfg["L"])
    ref = _ORACLE_CACHE[name + "/bwd"]
    for key in ("dQ", "dK", "dV"):
        amb = _ambiguous_rows(cfg, inp, key[1]) if key != "dV" else None
        err = _check_grad(to_numpy64(grads[key]), ref[key], "bf16", key, amb, cfg["L"])
        print(f"cfg5 flags={flags} {key}: max {err.max():.3e} mean {err.mean():.3e} "
              f"(rows with an ambiguous ReLU decision: {0 if amb is None else int(amb.sum())} of {amb.size if amb is not None else 0})")
    for key in ("dgate_w", "dgate_b", "domega"):
        err = small_vector_error(to_numpy64(grads[key]), ref[key])
        print(f"cfg5 flags={flags} {key}: max {err.max():.3e}")
        assert err.max() <= BF16_MAX, (key, err.max())
    db = float(grads["dbeta"].cpu()[0])
    rel = abs(db - ref["dbeta_closed"]) / abs(ref["dbeta_closed"])
    ref_O, ref_aux = _ORACLE_CACHE[name]
    dD = -(np.asarray(inp["dO"], dtype=np.float64) * ref_O).sum(-1) / ref_aux["D"]
    scale = 2.0 * 1e-6 * np.sqrt((dD ** 2).sum())   # see _dbeta_error
    err = abs(db - ref["dbeta_closed"]) / max(abs(ref["dbeta_closed"]), scale)
    print(f"cfg5 flags={flags} dbeta {db:.6e} ref {ref['dbeta_closed']:.6e} plain rel {rel:.3e} normalised {err:.3e}")
    assert err <= BF16_MAX, (db, ref["dbeta_closed"], err)


@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", 0), ("bf16", 1)])
def test_backward_at_the_configurations_epsilon(dtype, flags):
    """Backward with the denominator constant of the configurations (1e-6) instead of the larger one the
    small cases use: dbeta, which only acts through that constant, is then ~1e-6 of the other gradients."""
    import torch
    cfg = dict(B=2, H=2, n=1536, d=64, L=6, m=256 if dtype == "bf16" else 64, dtype=dtype)
    inp = wi.make_inputs(**cfg, seed=460, w_seed=461, gate_std=0.3, gate_seed=462, mean_shift=0.25, scale=0.7,
                         backward=True)
    ctx = _ctx(cfg, flags=flags)
    dev = device_inputs(inp, dtype)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    ctx.forward(*args)
    grads = ctx.backward(*args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _check_backward(cfg, inp, grads)


# ---------------------------------------------------------------- seeded random shapes
def _random_shapes(seed, count, backward):
    """Shapes drawn from a fixed seed: ragged n, every L, both feature counts, few and many slabs (so that
    a slab is cut into several chunks, or handled by one CTA without a reduction launch)."""
    import random
    rng = random.Random(seed)
    out = []
    for _ in range(count):
        m = rng.choice([128, 256])
        L = rng.randint(1, 8)
        B, H = rng.choice([(1, 1), (1, 3), (2, 2), (3, 5), (5, 1), (6, 7)] if backward else
                          [(1, 1), (1, 3), (2, 2), (3, 5), (9, 9), (20, 8), (2, 40)])
        nmax = (1500 if B * H <= 6 else 500) if backward else (5000 if B * H <= 10 else (1500 if B * H <= 40 else 700))
        out.append(dict(B=B, H=H, n=rng.randint(1 << L, nmax), d=64, L=L, m=m, gate_per_head=rng.choice([1, 1, 0])))
    return out


FWD_RANDOM = _random_shapes(11, 10, backward=False)
BWD_RANDOM = _random_shapes(12, 5, backward=True)


@pytest.mark.parametrize("case", range(len(FWD_RANDOM)))
def test_forward_random_shapes_tensor_core(case):
    import torch
    cfg = dict(FWD_RANDOM[case], dtype="bf16")
    inp = wi.make_inputs(**cfg, seed=5000 + case, w_seed=6000 + case, gate_std=0.3, gate_seed=7000 + case,
                         mean_shift=0.25, scale=0.7)
    ctx = _ctx(cfg)
    assert ctx.uses_tensor_cores()
    dev = device_inputs(inp, "bf16")
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    O = ctx.forward(*args).clone()
    O2 = ctx.forward(*args)
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    assert torch.equal(O, O2), "two runs on the same inputs differ"
    _check(to_numpy64(O), _oracle_forward(cfg, inp), "bf16", "O")


@pytest.mark.parametrize("case", range(len(BWD_RANDOM)))
def test_backward_random_shapes_tensor_core(case):
    import torch
    cfg = dict(BWD_RANDOM[case], dtype="bf16", eps=1e-3)
    inp = wi.make_inputs(**cfg, seed=8000 + case, w_seed=8100 + case, gate_std=0.3, gate_seed=8200 + case,
                         mean_shift=0.25, scale=0.7, backward=True)
    ctx = _ctx(cfg)
    dev = device_inputs(inp, "bf16")
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    ctx.forward(*args)
    grads = ctx.backward(*args, dev["dO"])
    torch.cuda.synchronize()
    assert ctx.query_status() == 0
    _check_backward(cfg, inp, grads)


# ---------------------------------------------------------------- a bounded wait that runs out
def test_bounded_wait_runs_out_and_is_reported_once():
    """The error path of the tensor-core kernels' waits, on a one-CTA self-test kernel: a wait limited to a
    millisecond on a barrier that is one arrival short gives up, the status word and the abort flag are set,
    the second role leaves through the abort flag, the kernel returns; the host sees WERSA_ERR_TIMEOUT once,
    then WERSA_OK, and the context still computes correctly afterwards."""
    import time
    import torch
    cfg = dict(B=1, H=1, n=256, d=64, L=3, m=128, dtype="bf16")
    inp = wi.make_inputs(**cfg, seed=3, w_seed=4)
    dev = device_inputs(inp, "bf16")
    ctx = _ctx(cfg)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    want = ctx.forward(*args).clone()
    assert ctx.query_status() == 0
    t0 = time.perf_counter()
    observed = ctx.selftest_wait_timeout(limit_us=1000)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 1.0          # the kernel returned by itself, well within a second
    assert observed.cpu().tolist() == [1, 0, 0]
    assert ctx.query_status() == 5                  # WERSA_ERR_TIMEOUT, reported once
    assert ctx.query_status() == 0
    assert torch.equal(ctx.forward(*args), want)
    assert ctx.query_status() == 0


# ---------------------------------------------------------------- error paths that need a device
def test_error_paths_on_device():
    import paper_2507_08637_b200 as wersa
    import torch
    cfg = dict(B=1, H=1, n=64, d=64, L=3, m=64, dtype="f32")
    inp = wi.make_inputs(**cfg, backward=True)
    dev = device_inputs(inp, "f32")
    ctx = _ctx(cfg)
    args = (dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    with pytest.raises(wersa.WersaError) as e:
        ctx.backward(*args, dev["dO"])
    assert e.value.status == 6
    # misaligned Q
    big = torch.zeros(dev["Q"].numel() + 1, device="cuda")
    with pytest.raises(wersa.WersaError) as e:
        ctx.forward(big[1:].view_as(dev["Q"]), *args[1:])
    assert e.value.status == 1
    fo = _ctx(cfg, flags=wersa.WERSA_FLAG_FORWARD_ONLY)
    fo.forward(*args)
    with pytest.raises(wersa.WersaError) as e:
        fo.backward(*args, dev["dO"])
    assert e.value.status == 2
