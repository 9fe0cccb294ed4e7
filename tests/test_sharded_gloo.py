"""Sequence-sharded forward, host side: two gloo ranks on CPU run paper_2507_08637_b200.sharded.forward_sharded
with a stand-in context whose four shard steps are the float64 oracle's pieces.  What is exchanged, when, and
that the shards' outputs put together equal the oracle's forward on the whole sequence is what this covers;
the kernels behind the real context are covered by the GPU parity tests."""
import os
import socket
from types import SimpleNamespace

import numpy as np

import wersa_inputs as wi
from oracle import wersa_oracle as orc

CFG = dict(B=2, H=3, n=200, d=8, L=3, m=16)
SPLIT = 128          # a multiple of 2^L: rank 0 takes rows [0, 128), rank 1 the rest
EPS = 1e-3


class OracleShardContext:
    """The interface forward_sharded uses, on CPU float64 tensors."""

    def __init__(self, n_local, L, gate_per_head):
        self.cfg = SimpleNamespace(seq_len=n_local)
        self.L, self.per_head = L, gate_per_head

    def shard_pool(self, Q, W, stream=None):
        import torch
        self.W = W.numpy()
        return torch.from_numpy(Q.numpy().sum(axis=2))

    def shard_gate(self, qsum_total, n_total, gate_w, gate_b, omega, stream=None):
        qbar = qsum_total.numpy() / float(n_total)
        # the oracle pools its argument: a one-token sequence equal to q-bar pools to q-bar
        _, self.f = orc.gate(qbar[:, :, None, :], gate_w.numpy(), gate_b.numpy(), omega.numpy(), self.L, self.per_head)

    def shard_keys(self, K, V, stream=None):
        import torch
        K, V = K.numpy(), V.numpy()
        B, H = K.shape[:2]
        m = self.W.shape[1]
        S, z = np.zeros((B, H, m, K.shape[3])), np.zeros((B, H, m))
        for b in range(B):
            for h in range(H):
                phi = orc.features(orc.haar_filter(K[b, h], self.f[b, h]), self.W)
                S[b, h], z[b, h] = phi.T @ V[b, h], phi.sum(axis=0)
        return torch.from_numpy(S), torch.from_numpy(z)

    def shard_output(self, Q, S_total, z_total, beta, out=None, stream=None):
        import torch
        Q, S, z = Q.numpy(), S_total.numpy(), z_total.numpy()
        O = np.zeros_like(Q)
        for b in range(Q.shape[0]):
            for h in range(Q.shape[1]):
                phi = orc.features(orc.haar_filter(Q[b, h], self.f[b, h]), self.W, float(beta[0]))
                O[b, h] = (phi @ S[b, h]) / (phi @ z[b, h] + EPS)[:, None]
        return torch.from_numpy(O)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _inputs(per_head):
    inp = wi.make_inputs(**CFG, seed=31, w_seed=32, gate_std=0.3, gate_seed=33, mean_shift=0.25, scale=0.7)
    return {k: np.asarray(v, dtype=np.float64) for k, v in inp.items()}


def _rank_main(rank, world, port, per_head, out):
    import torch
    import torch.distributed as dist
    from paper_2507_08637_b200.sharded import forward_sharded, total_length
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    inp = _inputs(per_head)
    rows = slice(0, SPLIT) if rank == 0 else slice(SPLIT, CFG["n"])
    t = lambda a: torch.from_numpy(np.ascontiguousarray(a))
    Q, K, V = (t(inp[k][:, :, rows]) for k in ("Q", "K", "V"))
    ctx = OracleShardContext(Q.shape[2], CFG["L"], per_head)
    assert total_length(Q.shape[2], "cpu") == CFG["n"]
    O = forward_sharded(ctx, Q, K, V, t(inp["W"]), t(inp["beta"]), t(inp["gate_w"]), t(inp["gate_b"]), t(inp["omega"]))
    out[rank] = O.numpy()
    dist.barrier()
    dist.destroy_process_group()


def _run(per_head):
    import torch.multiprocessing as mp
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, port, per_head, out), nprocs=world, join=True)
        res = dict(out)
    inp = _inputs(per_head)
    ref = orc.forward(inp["Q"], inp["K"], inp["V"], inp["W"], float(inp["beta"][0]), inp["gate_w"], inp["gate_b"],
                      inp["omega"], CFG["L"], eps=EPS, gate_per_head=per_head)
    got = np.concatenate([res[0], res[1]], axis=2)
    assert got.shape == ref.shape
    assert np.max(np.abs(got - ref)) < 1e-10 * max(1.0, np.max(np.abs(ref)))


def test_two_sequence_shards_give_the_whole_sequence_forward_per_head_gate():
    _run(1)


def test_two_sequence_shards_give_the_whole_sequence_forward_batch_wide_gate():
    _run(0)
