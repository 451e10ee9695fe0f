"""F-sliced tensor parallelism of the path-composed MoE layer (the second way the layer shards; token data
parallelism over replicas is in ``replicas.py``).

Rank g of G holds, of EVERY expert, the rows [f0, f1) of W_gate and W_up and the matching columns of W_down
(and the same slice of the shared expert).  SwiGLU acts element-wise along F and the projection is linear in
its input, so  y = sum_g y_g  with  y_g = the layer evaluated on rank g's slices: for a rank the layer is simply
a layer of width f1 - f0 on its own weight shard.  Routing and grouping depend on the logits only and are
replicated (integer-identical on every rank).  There is exactly one exchange step: the sum of the partial
outputs, as a reduce-scatter over token rows (each rank ends up with the complete y of its T/G tokens) or an
all-reduce.  The partial y of a rank is accumulated in its own memory by the stage-2 kernel first; the
collective is NCCL's (torch.distributed) and reads and writes local memory only.

Slices are aligned to the tile width of the tensor-core kernels (128 columns of F), so widths may differ by
one tile between ranks when F / 128 is not a multiple of G (F = 1408 is 11 tiles).
"""
from __future__ import annotations

import numpy as np

TILE_F = 128


def slice_bounds(F: int, G: int, g: int, tile: int = TILE_F):
    """[f0, f1) of rank g: the F / tile column tiles are dealt out in contiguous runs whose lengths differ by at
    most one (the first F/tile mod G ranks get the longer run).  F need not be a multiple of `tile`: the last
    tile is then the short one and belongs to the last rank."""
    if not (0 <= g < G) or F <= 0 or tile <= 0:
        raise ValueError("slice_bounds: need 0 <= g < G, F > 0, tile > 0")
    tiles = (F + tile - 1) // tile
    if G > tiles:
        raise ValueError(f"slice_bounds: {G} ranks but only {tiles} tiles of {tile} columns")
    base, extra = divmod(tiles, G)
    t0 = g * base + min(g, extra)
    t1 = t0 + base + (1 if g < extra else 0)
    return t0 * tile, min(t1 * tile, F)


def shard_expert_weights(w_gate, w_up, w_down, G: int, g: int, tile: int = TILE_F):
    """Rank g's contiguous shards of the routed experts: w_gate, w_up [n,F,H] -> [n,Fg,H]; w_down [n,H,F] ->
    [n,H,Fg].  Works on numpy arrays (any dtype, bf16 bit patterns included)."""
    f0, f1 = slice_bounds(w_gate.shape[1], G, g, tile)
    return (np.ascontiguousarray(w_gate[:, f0:f1, :]), np.ascontiguousarray(w_up[:, f0:f1, :]),
            np.ascontiguousarray(w_down[:, :, f0:f1]))


def shard_shared_weights(ws_gate, ws_up, ws_down, G: int, g: int, tile: int = TILE_F):
    """The same for the shared expert: [F_sh,H] -> [Fg,H]; [H,F_sh] -> [H,Fg]."""
    if ws_gate is None:
        return None, None, None
    f0, f1 = slice_bounds(ws_gate.shape[0], G, g, tile)
    return (np.ascontiguousarray(ws_gate[f0:f1, :]), np.ascontiguousarray(ws_up[f0:f1, :]),
            np.ascontiguousarray(ws_down[:, f0:f1]))


def token_shard(T: int, G: int, g: int):
    """Rows [t0, t1) of y that rank g owns after the reduce-scatter: equal shares of ceil(T/G) rows (the
    collective wants equal chunks; the last ranks' shares may be short or empty)."""
    per = (T + G - 1) // G
    return min(g * per, T), min((g + 1) * per, T)


def reduce_scatter_rows(y_partial, group=None):
    """Sums the partial outputs of all ranks and leaves every rank with its own token rows.

    y_partial: this rank's partial y [T,H] (torch tensor, fp32, on the rank's device; gloo: CPU).  Returns
    (y_rows, (t0, t1)): the complete rows [t0, t1) of y.  T is padded up to a multiple of the world size inside
    (zero rows), because the collective moves equal chunks."""
    import torch
    import torch.distributed as dist
    G = dist.get_world_size(group)
    g = dist.get_rank(group)
    T, H = y_partial.shape
    per = (T + G - 1) // G
    if per * G != T:
        pad = torch.zeros(per * G - T, H, dtype=y_partial.dtype, device=y_partial.device)
        y_partial = torch.cat([y_partial, pad], dim=0)
    out = torch.empty(per, H, dtype=y_partial.dtype, device=y_partial.device)
    if dist.get_backend(group) == "gloo":     # gloo has no reduce_scatter: all-reduce and keep the own rows
        buf = y_partial.clone()
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
        out.copy_(buf[g * per:(g + 1) * per])
    else:
        dist.reduce_scatter_tensor(out, y_partial.contiguous(), op=dist.ReduceOp.SUM, group=group)
    t0, t1 = token_shard(T, G, g)
    return out[: t1 - t0], (t0, t1)


def all_reduce_y(y_partial, group=None):
    """Sums the partial outputs in place: every rank ends up with the complete y [T,H]."""
    import torch.distributed as dist
    dist.all_reduce(y_partial, op=dist.ReduceOp.SUM, group=group)
    return y_partial
