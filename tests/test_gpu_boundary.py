"""Boundary behaviour of the C-ABI on the GPU: options that combine, knobs that are fixed when a plan is created,
and the give-up path of the kernels' bounded waits (a wait that runs out returns a status; nothing hangs or faults).
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu

TOL = 1e-5
SANITY = 5e-6


@pytest.fixture(scope="module")
def lib():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2002_03260_b200 as d
    return d


def _inputs():
    from paper_2002_03260_b200 import inputs
    return inputs


def _finish(plan):
    torch.cuda.synchronize()
    plan.status()


def test_inverse_solve_with_nodes_on_output(lib, oracle):
    """DFT3D_INVERSE_SOLVE | DFT3D_NODES_ON_OUTPUT: the system matrix is Eq. 1 read literally, V[k, n] = exp(-2 pi i
    w_k n) with arbitrary evaluation points w_k.  The solve plan undoes the forward plan of the same orientation and
    agrees with the oracle's LAPACK solve of that system."""
    shape = (64, 96, 128)
    rng = np.random.default_rng(203)
    nodes = [(np.arange(n) + 0.3 * rng.uniform(-1, 1, n)) / n for n in shape]
    nodes[2] = None
    x = _inputs().cube(shape, "normal", 204, device="cuda")
    fwd = lib.Plan(*shape, nodes=nodes, flags=lib.DFT3D_NODES_ON_OUTPUT)
    X = fwd(x)
    _finish(fwd)
    fwd.destroy()
    Xh = X.cpu().numpy()
    assert oracle.rel_l2(Xh, oracle.dft3d(x.cpu().numpy(), nodes=nodes, nodes_on_output=True)) < SANITY
    inv = lib.Plan(*shape, sign=lib.DFT3D_INVERSE, nodes=nodes,
                   flags=lib.DFT3D_INVERSE_SOLVE | lib.DFT3D_NODES_ON_OUTPUT)
    back = inv(X)
    _finish(inv)
    inv.destroy()
    assert oracle.rel_l2(back.cpu().numpy(), x.cpu().numpy()) < TOL
    want = oracle.solve3d(Xh.astype(np.complex128), nodes, nodes_on_output=True)
    assert oracle.rel_l2(back.cpu().numpy(), want) < SANITY
    # the solve of the other orientation is a different system
    other = lib.Plan(*shape, sign=lib.DFT3D_INVERSE, nodes=nodes, flags=lib.DFT3D_INVERSE_SOLVE)
    y = other(X)
    _finish(other)
    other.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), x.cpu().numpy()) > 1e-2


@pytest.mark.parametrize("split", ["fp16", "tf32"])
def test_auto_two_axes_with_destroy_input_keeps_a_workspace(lib, oracle, split):
    """DFT3D_AUTO over axes (1, 2) with nodes on axis 1 (KDFT) and a 512-point axis 2 (FFT): two passes,
    in -> workspace -> out.  DFT3D_DESTROY_INPUT must not turn the first pass into an in-place pass on the input
    (a KDFT pass re-reads its lines for every output tile), so the plan keeps a workspace of its own."""
    sf = lib.DFT3D_SPLIT_FP16 if split == "fp16" else lib.DFT3D_SPLIT_TF32
    shape = (8, 256, 512)
    nodes = [None, _inputs().sorted_nodes(shape, 206)[1], None]
    x = _inputs().cube(shape, "normal", 207, device="cuda")
    xh = x.cpu().numpy()
    want = oracle.dft_axis(oracle.dft_axis(xh.astype(np.complex128), 1, nodes=nodes[1]), 2)
    plan = lib.Plan(*shape, mode=lib.DFT3D_AUTO, nodes=nodes, flags=sf | lib.DFT3D_DESTROY_INPUT, axes=(1, 2))
    assert plan.workspace_bytes == x.numel() * 8
    y = plan(x)
    _finish(plan)
    plan.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), want) < SANITY


def test_knobs_are_fixed_when_the_plan_is_created(lib, monkeypatch):
    """Tuning knobs come from the environment at plan creation and live in the plan: changing the environment
    afterwards changes neither the launches nor one bit of the output."""
    shape = (256, 256, 256)
    x = _inputs().cube(shape, "normal", 208, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    first = plan(x).clone()
    launches = plan.launches
    _finish(plan)
    for name, value in (("DFT3D_FFT_INPLACE", "1"), ("DFT3D_FFT_L2_PREFETCH", "0"), ("DFT3D_TEST_SILENT_PRODUCER", "1")):
        monkeypatch.setenv(name, value)
    again = plan(x)
    _finish(plan)
    assert plan.launches == launches and torch.equal(first, again)
    plan.destroy()
    for name in ("DFT3D_TEST_SILENT_PRODUCER",):
        monkeypatch.delenv(name)
    # a plan created now does see the knobs (the in-place schedule owns no workspace) and computes the same transform
    changed = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    other = changed(x)
    _finish(changed)
    changed.destroy()
    num = float(((other.to(torch.complex128) - first.to(torch.complex128)).abs() ** 2).sum())
    den = float((first.to(torch.complex128).abs() ** 2).sum())
    assert (num / den) ** 0.5 < SANITY


@pytest.mark.parametrize("mode_name,shape,axes", [("kdft", (64, 64, 64), None), ("kdft_tf32", (64, 64, 64), None),
                                                 ("fft", (64, 64, 256), (2,)), ("fft", (256, 64, 64), (0,))])
def test_bounded_waits_give_up_and_report(lib, oracle, monkeypatch, mode_name, shape, axes):
    """Every device-side wait has a clock budget.  Here the budget is about a millisecond and the TMA producer of every
    CTA stays silent, so nothing is ever in flight and every role's first wait runs out: the kernels return by
    themselves, the plan reports DFT3D_ERR_DEVICE_TIMEOUT, and the device is fine: a fresh plan right after matches
    the oracle."""
    monkeypatch.setenv("DFT3D_TEST_SILENT_PRODUCER", "1")
    monkeypatch.setenv("DFT3D_WAIT_LIMIT_CLOCKS", "2000000")
    mode = lib.DFT3D_FFT if mode_name == "fft" else lib.DFT3D_KDFT
    flags = lib.DFT3D_SPLIT_TF32 if mode_name == "kdft_tf32" else 0
    x = _inputs().cube(shape, "normal", 209, device="cuda")
    silent = lib.Plan(*shape, mode=mode, flags=flags, axes=axes)
    monkeypatch.delenv("DFT3D_TEST_SILENT_PRODUCER")
    monkeypatch.delenv("DFT3D_WAIT_LIMIT_CLOCKS")
    silent(x)
    torch.cuda.synchronize()
    with pytest.raises(lib.Dft3dError) as e:
        silent.status()
    assert e.value.status == 5
    silent.destroy()
    plan = lib.Plan(*shape, mode=mode, flags=flags, axes=axes)
    y = plan(x)
    _finish(plan)
    plan.destroy()
    want = x.cpu().numpy().astype(np.complex128)
    for a in (axes or (0, 1, 2)):
        want = oracle.dft_axis(want, a)
    assert oracle.rel_l2(y.cpu().numpy(), want) < SANITY


def test_fft_split_option_and_query(lib):
    """fft_split names the factor pair {N1, N2} of Eq. 17 per axis.  The kernels realise one pair per length; that pair
    is accepted (and is what {0, 0} selects), any other is refused, and the plan reports the pair it uses."""
    shape = (256, 512, 256)
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, fft_split=[(16, 16), (32, 16), None])
    assert [plan.fft_split(a) for a in range(3)] == [(16, 16), (32, 16), (16, 16)]
    plan.destroy()
    for bad in ([(8, 32), None, None], [None, (16, 32), None], [None, None, (16, 8)]):
        with pytest.raises(lib.Dft3dError) as e:
            lib.Plan(*shape, mode=lib.DFT3D_FFT, fft_split=bad)
        assert e.value.status == 2
    kd = lib.Plan(64, 64, 64)
    with pytest.raises(lib.Dft3dError) as e:
        kd.fft_split(0)
    assert e.value.status == 1
    kd.destroy()


@pytest.mark.parametrize("sign", [-1, +1])
def test_ring_blocks_of_axis0_on_the_gpu_kernels(lib, oracle, sign):
    """The per-rank block product of the one-shuffle ring (a square nonuniform-node plan per source rank and a phase
    on the input rows) is a function of (rank, source rank) alone: summing it over the source ranks, rank by rank in
    this one process with no exchange, must give each rank's slab of the axis-0 transform."""
    from paper_2002_03260_b200 import sharded
    n0, n1, n2, world = 256, 64, 64, 4
    b = n0 // world
    x = _inputs().cube((n0, n1, n2), "normal", 210, device="cuda")
    want = oracle.dft_axis(x.cpu().numpy().astype(np.complex128), 0, sign=sign, scale=(1.0 / n0 if sign > 0 else 1.0))
    for rank in (0, 3):
        _, block_product = sharded.gpu_transforms(n0, n1, n2, rank, world, "kdft", sign=sign)
        acc = None
        for src in range(world):
            part = block_product(x[src * b:(src + 1) * b].contiguous(), src)
            acc = part if acc is None else acc + part
        torch.cuda.synchronize()
        assert oracle.rel_l2(acc.cpu().numpy(), want[rank * b:(rank + 1) * b]) < SANITY
