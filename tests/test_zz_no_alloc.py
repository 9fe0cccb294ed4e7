"""wersa_gate_static: the allocation-free variant of the mean-pool + gate step.

Some callers cannot allocate device memory where they need the gate (their allocator is frozen
or belongs to another framework, or device memory is fully committed), so this entry point keeps
its intermediate sums in a fixed array inside the library instead of a caller workspace.  The test
calls it through the C ABI twice in a row (the array keeps the previous call's contents, and the
second call must not be disturbed by them) and compares both results with what the regular
entry point, wersa_forward, leaves in its workspace.  Collected last on purpose."""
import numpy as np
import pytest

import wersa_inputs as wi
from tests.util import device_inputs, to_numpy64

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,per_head", [("bf16", 1), ("f32", 0)])
def test_gate_static_matches_forward_twice(dtype, per_head):
    import paper_2507_08637_b200 as wersa
    import torch
    cfg = dict(B=2, H=3, n=2304, d=64, L=5, m=64, dtype=dtype, gate_per_head=per_head)
    inp = wi.make_inputs(**cfg, seed=21, w_seed=22, gate_std=0.3, gate_seed=23, mean_shift=0.3)
    dev = device_inputs(inp, dtype)
    ctx = wersa.wersa_create(cfg["B"], cfg["H"], cfg["n"], cfg["d"], cfg["L"], cfg["m"], dtype=dtype,
                             gate_per_head=per_head)
    ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
    want_qbar, want_f = to_numpy64(ctx.saved("qbar")), to_numpy64(ctx.saved("f"))
    c = ctx.cfg
    qbar = torch.empty((cfg["B"] * cfg["H"], cfg["d"]), dtype=torch.float32, device="cuda")
    f = torch.empty((cfg["B"] * cfg["H"], cfg["L"] + 1), dtype=torch.float32, device="cuda")
    # a different problem first, so that the shared array holds foreign contents
    other = (dev["Q"].float() * 3.0 + 1.0).to(dev["Q"].dtype)
    wersa.wersa_gate_static(c, other, dev["gate_w"], dev["gate_b"], dev["omega"], qbar, f)
    torch.cuda.synchronize()
    assert np.abs(to_numpy64(f).reshape(want_f.shape) - want_f).max() > 1e-3
    for _ in range(2):
        qbar.fill_(float("nan"))
        f.fill_(float("nan"))
        wersa.wersa_gate_static(c, dev["Q"], dev["gate_w"], dev["gate_b"], dev["omega"], qbar, f)
        torch.cuda.synchronize()
        assert np.max(np.abs(to_numpy64(qbar).reshape(want_qbar.shape) - want_qbar)) <= 2e-6
        assert np.max(np.abs(to_numpy64(f).reshape(want_f.shape) - want_f)) <= 2e-6


def test_gate_static_calls_of_different_shapes_in_any_order():
    """A large layout, then a smaller one, then the large one again: the arrival counters sit at a fixed
    place at the end of the shared array, so that the sums and sigmoids one call leaves behind can never be
    mistaken for counters by the next, whatever its shape.  Each call is compared with what wersa_forward
    leaves in its own workspace for the same problem."""
    import paper_2507_08637_b200 as wersa
    import torch
    shapes = [dict(B=1, H=8, n=16384, d=64, L=8, m=64, dtype="bf16", gate_per_head=1),   # 74 chunks per slab
              dict(B=1, H=1, n=1024, d=64, L=3, m=64, dtype="f32", gate_per_head=1),     # one slab, 8 chunks
              dict(B=4, H=6, n=700, d=64, L=4, m=64, dtype="bf16", gate_per_head=0)]     # batch counters too
    want, devs, cfgs = [], [], []
    for i, cfg in enumerate(shapes):
        inp = wi.make_inputs(**cfg, seed=31 + i, w_seed=41 + i, gate_std=0.3, gate_seed=51 + i, mean_shift=0.3)
        dev = device_inputs(inp, cfg["dtype"])
        ctx = wersa.wersa_create(cfg["B"], cfg["H"], cfg["n"], cfg["d"], cfg["L"], cfg["m"], dtype=cfg["dtype"],
                                 gate_per_head=cfg["gate_per_head"])
        ctx.forward(dev["Q"], dev["K"], dev["V"], dev["W"], dev["beta"], dev["gate_w"], dev["gate_b"], dev["omega"])
        want.append((to_numpy64(ctx.saved("qbar")), to_numpy64(ctx.saved("f"))))
        devs.append(dev)
        cfgs.append(ctx.cfg)
    for i in (0, 1, 0, 2, 1, 2, 0):
        cfg, dev = shapes[i], devs[i]
        qbar = torch.full((cfg["B"] * cfg["H"], cfg["d"]), float("nan"), dtype=torch.float32, device="cuda")
        f = torch.full((cfg["B"] * cfg["H"], cfg["L"] + 1), float("nan"), dtype=torch.float32, device="cuda")
        wersa.wersa_gate_static(cfgs[i], dev["Q"], dev["gate_w"], dev["gate_b"], dev["omega"], qbar, f)
        torch.cuda.synchronize()
        assert np.max(np.abs(to_numpy64(qbar).reshape(want[i][0].shape) - want[i][0])) <= 2e-6, i
        assert np.max(np.abs(to_numpy64(f).reshape(want[i][1].shape) - want[i][1])) <= 2e-6, i


def test_gate_static_rejects_problems_beyond_its_fixed_scratch():
    import paper_2507_08637_b200 as wersa
    import torch
    # 8192 slabs x (64 + 3) floats > 253952 floats
    cfg = wersa.make_config(128, 64, 64, 64, 2, 64, dtype="f32")
    Q = torch.zeros(16, device="cuda")
    om = torch.ones(3, device="cuda")
    out = torch.zeros(8, device="cuda")
    with pytest.raises(wersa.WersaError) as e:
        wersa.wersa_gate_static(cfg, Q, None, None, om, out, out)
    assert e.value.status == 7
