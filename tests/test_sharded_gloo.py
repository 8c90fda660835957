"""One cube spread over several ranks (slabs of n0-planes; axis 0 across the ranks by the ring of Algorithm 1 or by one
re-partition), run as CPU processes over gloo (127.0.0.1).  The exchange and index logic is what is under test: the
per-rank transforms are stand-ins typed here from the definitions (numpy), and the assembled result is compared with
the float64 oracle's transform of the whole cube."""
import os
import socket

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _dft_matrix(rows, cols, n, sign):
    """M[k, j] = exp(sign 2 pi i k j / n) for the given row and column indices (Eq. 14's kernel)."""
    return np.exp(sign * 2j * np.pi * np.outer(rows, cols) / n)


def _worker(rank, world, port, shape, sign, route, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2002_03260_b200 import inputs, sharded
    n0, n1, n2 = shape
    x = inputs.cube(shape, "normal", 4242, device="cpu")          # every rank draws the same cube and keeps its slab
    lo, hi = sharded.slab_range(n0, rank, world)
    slab = x[lo:hi].to(torch.complex128).contiguous()
    keep = slab.clone()
    b = hi - lo

    def local_axes12(s):
        a = s.numpy()
        a = np.einsum("kj,ajc->akc", _dft_matrix(np.arange(n1), np.arange(n1), n1, sign), a)
        a = np.einsum("kj,abj->abk", _dft_matrix(np.arange(n2), np.arange(n2), n2, sign), a)
        return torch.from_numpy(np.ascontiguousarray(a))

    def block_product(block, src):
        M = _dft_matrix(np.arange(lo, hi), np.arange(src * b, (src + 1) * b), n0, sign)   # rows of this rank, columns of src
        return torch.from_numpy(np.ascontiguousarray(np.einsum("kj,jbc->kbc", M, block.numpy())))

    def axis0_transform(columns):
        M = _dft_matrix(np.arange(n0), np.arange(n0), n0, sign)
        return torch.from_numpy(np.ascontiguousarray(np.einsum("kj,jbc->kbc", M, columns.numpy())))

    y = sharded.transform_sharded(slab, local_axes12, block_product if route == "one_shuffle" else axis0_transform, route)
    assert torch.equal(slab, keep)                                 # the caller's slab is only read
    gathered = [None] * world
    dist.all_gather_object(gathered, (rank, y.numpy()))
    if rank == 0:
        full = np.concatenate([g[1] for g in sorted(gathered, key=lambda g: g[0])], axis=0)
        out.put((x.numpy(), full))
    dist.barrier()
    dist.destroy_process_group()


@pytest.mark.parametrize("world,route,shape,sign", [(2, "one_shuffle", (8, 6, 10), -1), (3, "one_shuffle", (6, 4, 8), +1),
                                                   (2, "repartition", (8, 6, 10), -1), (4, "repartition", (8, 8, 6), +1)])
def test_sharded_transform_matches_the_oracle(oracle, world, route, shape, sign):
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, shape, sign, route, out)) for r in range(world)]
    for p in procs:
        p.start()
    x, got = out.get(timeout=180)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    want = oracle.dft3d(x, sign=sign)
    assert oracle.rel_l2(got, want) < 1e-12


def test_slab_range_and_refusals():
    from paper_2002_03260_b200 import sharded
    assert [sharded.slab_range(12, r, 3) for r in range(3)] == [(0, 4), (4, 8), (8, 12)]
    with pytest.raises(ValueError):
        sharded.slab_range(10, 0, 3)
