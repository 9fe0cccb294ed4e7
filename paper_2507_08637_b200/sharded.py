"""Sequence-sharded forward: every rank holds a contiguous shard of each slab's sequence (all shards but the
last a multiple of 2^levels tokens) and runs the library's four shard steps; the two sums in between (column
sums of Q, then S' and z') are all-reduces over the ranks.  torch.distributed does the exchange, the library's
kernels do every step of the arithmetic."""
import torch


def allreduce_sum_(tensors, group=None):
    """In-place sum over the ranks of `group` (no-op without an initialised process group)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return tensors
    for t in tensors:
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)
    return tensors


def total_length(n_local, device, group=None):
    """Whole sequence length: the sum of the shards' lengths."""
    t = torch.tensor([int(n_local)], dtype=torch.int64, device=device)
    allreduce_sum_([t], group)
    return int(t.item())


def forward_sharded(ctx, Q, K, V, W, beta, gate_w, gate_b, omega, out=None, group=None, n_total=None, stream=None):
    """ctx: a WersaContext created with seq_len = this rank's shard length.  Q, K, V: this rank's shards.
    Returns this rank's shard of O."""
    if n_total is None:
        n_total = total_length(ctx.cfg.seq_len, Q.device, group)
    qsum = ctx.shard_pool(Q, W, stream=stream)
    allreduce_sum_([qsum], group)
    ctx.shard_gate(qsum, n_total, gate_w, gate_b, omega, stream=stream)
    S, z = ctx.shard_keys(K, V, stream=stream)
    S_total, z_total = S.clone(), z.clone()
    allreduce_sum_([S_total, z_total], group)
    return ctx.shard_output(Q, S_total, z_total, beta, out=out, stream=stream)


def backward_sharded(ctx, Q, K, V, W, beta, gate_w, gate_b, omega, dO, group=None, n_total=None, stream=None):
    """Backward of forward_sharded on the same context (call it after forward_sharded with the same shards).
    Returns dict(dQ, dK, dV, dbeta, dgate_w, dgate_b, domega): dQ, dK, dV are this rank's shards, the parameter
    gradients are those of the whole sequence (the same on every rank).  Three sums cross the ranks: dS' and dz',
    then the band inner products together with the sum of dD'."""
    if n_total is None:
        n_total = total_length(ctx.cfg.seq_len, Q.device, group)
    dS, dz = ctx.shard_backward_queries(Q, beta, dO, stream=stream)
    dS_total, dz_total = dS.clone(), dz.clone()
    allreduce_sum_([dS_total, dz_total], group)
    dK, dV, df, sumdD = ctx.shard_backward_keys(K, V, dS_total, dz_total, stream=stream)
    df_total, sumdD_total = df.clone(), sumdD.clone()
    allreduce_sum_([df_total, sumdD_total], group)
    grads = ctx.shard_backward_gate(Q, df_total, sumdD_total, n_total, beta, gate_w, omega, stream=stream)
    grads.update(dK=dK, dV=dV)
    return grads
