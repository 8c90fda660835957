"""One cube spread over several ranks: slabs of n0-planes, axis 0 transformed across the ranks.

Rank r of G holds the planes [r*b, (r+1)*b) of an n0 x n1 x n2 cube, b = n0 / G.  Axes 1 and 2 are local to a slab (no
exchange).  Axis 0 needs every plane, and there are the two ways the paper describes (Section IV):

* the ring of Algorithm 1 ("one shuffle", for the KDFT formulation): the output slab of rank r is
  sum over source ranks s of M_0[rows of r, columns of s] * slab_s.  Every rank multiplies the slab it holds by the
  matching block of the axis-0 matrix, adds the product to its output, and passes the slab on to its neighbour; after
  G - 1 shuffles every slab has visited every rank.  The exchange of step i can travel while the product of step i
  runs: the slab in hand is only read.
* one re-partition (for the FFT formulation, Section IV-D's gather): an all-to-all turns slabs of n0-planes into
  slabs of n1-rows that hold all of axis 0, the axis is transformed locally, and a second all-to-all turns them back.

The exchanges are torch.distributed point-to-point operations and all-to-alls (NCCL on GPUs, gloo on CPUs), received
blocks land in this rank's own memory before any kernel reads them.  The per-rank transforms are callables, so the same
orchestration runs with the library's plans on GPUs (`gpu_transforms`) and with any stand-in on CPUs (the tests).
"""
import math

import torch
import torch.distributed as dist


def slab_range(n0, rank, world):
    """Planes [lo, hi) of rank `rank`; the slabs have equal size (n0 must be a multiple of the world size)."""
    if n0 % world != 0:
        raise ValueError("n0 = %d is not a multiple of the world size %d" % (n0, world))
    b = n0 // world
    return rank * b, (rank + 1) * b


def _ring_exchange(send, recv, rank, world, group):
    """Every rank sends `send` to rank+1 and receives `recv` from rank-1 (the source/target pairs of Algorithm 1)."""
    ops = [dist.P2POp(dist.isend, send, (rank + 1) % world, group=group),
           dist.P2POp(dist.irecv, recv, (rank - 1) % world, group=group)]
    return dist.batch_isend_irecv(ops)


def one_shuffle_axis0(slab, block_product, group=None):
    """Algorithm 1 along axis 0.  `slab`: this rank's planes [b, n1, n2], complex.  `block_product(block, src)` returns
    M_0[rows of this rank, columns of rank src] applied along axis 0 of `block` (same shape).  Returns this rank's slab
    of the result.  G - 1 shuffles; the exchange of a step is in flight while that step's product runs."""
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    out = None
    hand, src = slab, rank
    spare = torch.empty_like(slab) if world > 1 else None
    for step in range(world):
        last = step == world - 1
        reqs = [] if last else _ring_exchange(hand, spare, rank, world, group)
        # the slab in hand is multiplied while it travels on to the neighbour (both only read it)
        part = block_product(hand, src)
        out = part if out is None else out + part
        if last:
            break
        for r in reqs:
            r.wait()
        if hand is slab:
            hand, spare = spare, torch.empty_like(slab)   # the caller's slab is never written
        else:
            hand, spare = spare, hand
        src = (src - 1) % world
    return out


def repartition_axis0(slab, axis0_transform, group=None):
    """The all-to-all route along axis 0.  `slab`: [b, n1, n2]; n1 must be a multiple of the world size.
    `axis0_transform(columns)` transforms axis 0 of a [n0, n1 / G, n2] tensor.  Returns this rank's slab of the result."""
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    b, n1, n2 = slab.shape
    if n1 % world != 0:
        raise ValueError("n1 = %d is not a multiple of the world size %d" % (n1, world))
    c = n1 // world
    # piece d of the send buffer: my planes, the n1-rows of rank d
    send = slab.reshape(b, world, c, n2).permute(1, 0, 2, 3).contiguous()
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    columns = recv.reshape(world * b, c, n2)               # piece s holds the planes of rank s: all of axis 0
    columns = axis0_transform(columns)
    send = columns.reshape(world, b, c, n2).contiguous()   # piece d: the output planes of rank d
    dist.all_to_all_single(recv, send, group=group)
    return recv.permute(1, 0, 2, 3).reshape(b, n1, n2).contiguous()


def transform_sharded(slab, local_axes12, axis0, route, group=None):
    """The whole 3D transform of a cube held in slabs: axes 1 and 2 locally (`local_axes12(slab)`), then axis 0 by
    `route` = "one_shuffle" (axis0 = block_product) or "repartition" (axis0 = axis0_transform)."""
    y = local_axes12(slab)
    if route == "one_shuffle":
        return one_shuffle_axis0(y, axis0, group)
    if route == "repartition":
        return repartition_axis0(y, axis0, group)
    raise ValueError("route must be 'one_shuffle' or 'repartition'")


def gpu_transforms(n0, n1, n2, rank, world, mode, sign=-1):
    """The per-rank callables on a GPU, built from the library's plans.

    local_axes12: a plan over axes (1, 2) of the [b, n1, n2] slab.
    KDFT -> block_product for the ring: the block M_0[r*b + k, s*b + j] = exp(sign 2 pi i (r*b + k)(s*b + j) / n0),
    k, j < b, is the b x b matrix of the nodes t_j = (s*b + j)/n0 (integer k) times the phase exp(sign 2 pi i r*b*t_j)
    of input row j: one plan per source rank (nodes on axis 0 of a [b, n1, n2] slab) and one multiplication of the rows
    by that phase.
    FFT -> axis0_transform for the re-partition: a plan over axis 0 of [n0, n1 / G, n2]."""
    from . import dft3d as lib
    b = n0 // world
    m = lib.DFT3D_KDFT if mode == "kdft" else lib.DFT3D_FFT
    p12 = lib.Plan(b, n1, n2, mode=m, sign=sign, axes=(1, 2))

    def local_axes12(slab):
        return p12(slab)

    if mode == "kdft":
        import numpy as np
        plans, phases = {}, {}

        def block_product(block, src):
            if src not in plans:
                t = (src * b + np.arange(b)) / float(n0)
                flags = lib.DFT3D_UNSCALED_INVERSE if sign > 0 else 0
                plans[src] = lib.Plan(b, n1, n2, mode=lib.DFT3D_KDFT, sign=sign, nodes=(t, None, None), axes=(0,),
                                      flags=flags)
                ang = sign * 2.0 * math.pi * ((rank * b * (src * b + np.arange(b))) % n0) / float(n0)
                scale = (1.0 / n0) if sign > 0 else 1.0
                phases[src] = torch.from_numpy((scale * np.exp(1j * ang)).astype(np.complex64)).to(block.device)
            return plans[src](block * phases[src][:, None, None])

        return local_axes12, block_product
    p0 = lib.Plan(n0, n1 // world, n2, mode=m, sign=sign, axes=(0,))

    def axis0_transform(columns):
        return p0(columns)

    return local_axes12, axis0_transform
