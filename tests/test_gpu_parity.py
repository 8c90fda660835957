"""Parity of the CUDA path (through the C-ABI) with the float64 oracle on the same seeded inputs.

Tolerance: relative L2 error <= 1e-5 against the float64 oracle (the bar the task states).  The
3xTF32 arithmetic with accumulation chains of 48 MMAs lands near 1e-6 per axis (the tensor core adds
into its fp32 accumulator with truncation, a bias that adds up over the axes), so tighter sanity
bounds are asserted as well: 2e-6 for one axis, 5e-6 for a 3D transform.  An error of ~2.6e-4 would
mean a split product is missing, >1e-3 an indexing bug.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu

TOL = 1e-5
SANITY = 5e-6       # one 3D transform (three axis passes)
SANITY_AXIS = 2e-6  # one axis pass


@pytest.fixture(scope="module")
def lib():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2002_03260_b200 as d
    return d


@pytest.fixture(autouse=True)
def _release_cached_blocks():
    """The library allocates its workspaces with cudaMalloc, outside torch's caching allocator: blocks torch keeps
    cached after a test with large tensors would be missing for the next test's plans (config 5 needs 128 GiB)."""
    yield
    if torch.cuda.is_available():
        import gc
        gc.collect()
        torch.cuda.empty_cache()


def _inputs():
    from paper_2002_03260_b200 import inputs
    return inputs


def _finish(plan):
    torch.cuda.synchronize()
    plan.status()


SPLITS = ["fp16", "tf32"]   # the two operand splits of the KDFT kernels; fp16 is the default where sizes allow


def _split_flag(lib, split):
    return lib.DFT3D_SPLIT_FP16 if split == "fp16" else lib.DFT3D_SPLIT_TF32


def _pre(lib, plan, kdft=True):
    """Launches before the axis passes: the fp16 split of the KDFT kernels first reduces the input to its largest
    magnitude (the FFT kernels scale line by line inside the pass)."""
    return 1 if (kdft and plan.split == lib.DFT3D_SPLIT_FP16) else 0


# ------------------------------------------------------------------ single axes (each kernel variant alone)

@pytest.mark.parametrize("shape", [(64, 64, 64), (64, 128, 192), (128, 64, 256), (192, 64, 64)])
@pytest.mark.parametrize("axis", [0, 1, 2])
@pytest.mark.parametrize("split", SPLITS)
def test_kdft_single_axis(lib, oracle, shape, axis, split):
    x = _inputs().cube(shape, "normal", 7 + axis, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_KDFT, flags=_split_flag(lib, split))
    assert plan.split == _split_flag(lib, split)
    y = plan.execute_axis(axis, x)
    _finish(plan)
    ref = oracle.dft_axis(x.cpu().numpy().astype(np.complex128), axis)
    err = oracle.rel_l2(y.cpu().numpy(), ref)
    assert err < SANITY_AXIS, (shape, axis, err)
    plan.destroy()


# ------------------------------------------------------------------ config 1: 64^3 KDFT forward, U(-1,1)

@pytest.mark.parametrize("split", SPLITS)
def test_config1_kdft_64(lib, oracle, split):
    shape = (64, 64, 64)
    x = _inputs().cube(shape, "uniform", 1001, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_KDFT, sign=lib.DFT3D_FORWARD, flags=_split_flag(lib, split))
    y = plan(x)
    _finish(plan)
    ref = oracle.dft3d(x.cpu().numpy())
    err = oracle.rel_l2(y.cpu().numpy(), ref)
    assert err < TOL and err < SANITY, err
    # the input is never written
    assert torch.equal(x, _inputs().cube(shape, "uniform", 1001, device="cuda"))
    plan.destroy()


@pytest.mark.parametrize("shape", [(64, 128, 256), (256, 64, 128), (128, 192, 64)])
@pytest.mark.parametrize("split", SPLITS)
def test_kdft_noncubic(lib, oracle, shape, split):
    x = _inputs().cube(shape, "uniform", 31, device="cuda")
    plan = lib.Plan(*shape, flags=_split_flag(lib, split))
    y = plan(x)
    _finish(plan)
    err = oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy()))
    assert err < SANITY, (shape, err)
    plan.destroy()


@pytest.mark.parametrize("split", SPLITS)
def test_kdft_workspace_groups(lib, oracle, split):
    """A small workspace limit forces the plane-group schedule (several launches per axis)."""
    shape = (64, 64, 128)
    x = _inputs().cube(shape, "normal", 32, device="cuda")
    plan = lib.Plan(*shape, workspace_limit=16 * 64 * 128 * 8, flags=_split_flag(lib, split))
    assert plan.workspace_bytes == 16 * 64 * 128 * 8 and plan.launches == _pre(lib, plan) + 1 + 2 * 4
    y = plan(x)
    _finish(plan)
    err = oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy()))
    assert err < SANITY, err
    plan.destroy()


@pytest.mark.parametrize("split", SPLITS)
def test_kdft_inverse_and_roundtrip(lib, oracle, split):
    shape = (128, 64, 64)
    x = _inputs().cube(shape, "normal", 33, device="cuda")
    sf = _split_flag(lib, split)
    fwd, inv = lib.Plan(*shape, sign=lib.DFT3D_FORWARD, flags=sf), lib.Plan(*shape, sign=lib.DFT3D_INVERSE, flags=sf)
    X = fwd(x)
    back = inv(X)
    _finish(inv)
    fwd.status()
    assert oracle.rel_l2(back.cpu().numpy(), x.cpu().numpy()) < TOL   # two transforms in a row
    ref = oracle.dft3d(X.cpu().numpy(), sign=+1, scaled_inverse=True)
    assert oracle.rel_l2(back.cpu().numpy(), ref) < SANITY
    raw = lib.Plan(*shape, sign=lib.DFT3D_INVERSE, flags=lib.DFT3D_UNSCALED_INVERSE | sf)
    y = raw(X)
    _finish(raw)
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(X.cpu().numpy(), sign=+1)) < SANITY
    for p in (fwd, inv, raw):
        p.destroy()


# ------------------------------------------------------------------ config 4: nonuniform KDFT 256^3

@pytest.mark.parametrize("split", SPLITS)
def test_config4_nonuniform_256(lib, oracle, split):
    shape = (256, 256, 256)
    inp = _inputs()
    x = inp.cube(shape, "normal", 1004, device="cuda")
    nodes = inp.sorted_nodes(shape, 2004)
    plan = lib.Plan(*shape, nodes=nodes, flags=_split_flag(lib, split))
    y = plan(x)
    _finish(plan)
    ref = oracle.dft3d(x.cpu().numpy(), nodes=nodes)
    err = oracle.rel_l2(y.cpu().numpy(), ref)
    assert err < TOL and err < SANITY, err
    plan.destroy()


def test_nonuniform_nodes_on_output_and_mixed(lib, oracle):
    shape = (64, 128, 64)
    inp = _inputs()
    x = inp.cube(shape, "normal", 41, device="cuda")
    nodes = inp.sorted_nodes(shape, 42)
    plan = lib.Plan(*shape, nodes=nodes, flags=lib.DFT3D_NODES_ON_OUTPUT)
    y = plan(x)
    _finish(plan)
    ref = oracle.dft3d(x.cpu().numpy(), nodes=nodes, nodes_on_output=True)
    assert oracle.rel_l2(y.cpu().numpy(), ref) < SANITY
    plan.destroy()
    mixed = (None, nodes[1], None)
    plan = lib.Plan(*shape, nodes=mixed)
    y = plan(x)
    _finish(plan)
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy(), nodes=mixed)) < SANITY
    plan.destroy()


# ------------------------------------------------------------------ config 2: 512^3 forward + inverse

@pytest.mark.slow
def test_config2_kdft_512_forward_inverse(lib, oracle):
    shape = (512, 512, 512)
    x = _inputs().cube(shape, "normal", 1002, device="cuda")
    fwd, inv = lib.Plan(*shape, sign=lib.DFT3D_FORWARD), lib.Plan(*shape, sign=lib.DFT3D_INVERSE)
    X = fwd(x)
    _finish(fwd)
    xh = x.cpu().numpy()
    ref = oracle.dft3d(xh)            # full float64 oracle: 2e11 complex MACs
    err = oracle.rel_l2(X.cpu().numpy(), ref)
    del ref
    assert err < TOL and err < SANITY, err
    back = inv(X)
    _finish(inv)
    assert oracle.rel_l2(back.cpu().numpy(), xh) < TOL
    fwd.destroy()
    inv.destroy()


# ------------------------------------------------------------------ host-buffer entry point

def test_execute_host(lib, oracle):
    shape = (64, 64, 128)
    x = _inputs().cube(shape, "uniform", 51, device="cpu").pin_memory()
    out = torch.empty_like(x).pin_memory()
    plan = lib.Plan(*shape)
    plan.execute_host(x, out)
    err = oracle.rel_l2(out.numpy(), oracle.dft3d(x.numpy()))
    assert err < SANITY, err
    plan.destroy()


# ------------------------------------------------------------------ FFT formulation (fused GEMM - twiddle - GEMM kernel)

@pytest.mark.parametrize("shape,axis", [((256, 256, 256), 0), ((256, 256, 256), 1), ((256, 256, 256), 2),
                                        ((256, 256, 1024), 2), ((256, 1024, 256), 1), ((1024, 256, 256), 0)])
@pytest.mark.parametrize("split", SPLITS)
def test_fft_single_axis(lib, oracle, shape, axis, split):
    x = _inputs().cube(shape, "normal", 61 + axis, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, flags=_split_flag(lib, split))
    assert plan.split == _split_flag(lib, split)
    y = plan.execute_axis(axis, x)
    _finish(plan)
    ref = oracle.dft_axis(x.cpu().numpy().astype(np.complex128), axis)
    err = oracle.rel_l2(y.cpu().numpy(), ref)
    assert err < SANITY_AXIS, (shape, axis, err)
    plan.destroy()


@pytest.mark.parametrize("split", SPLITS)
def test_fft_256_forward_inverse_and_kdft_agreement(lib, oracle, split):
    shape = (256, 256, 256)
    sf = _split_flag(lib, split)
    x = _inputs().cube(shape, "uniform", 62, device="cuda")
    fft = lib.Plan(*shape, mode=lib.DFT3D_FFT, flags=sf)
    kdft = lib.Plan(*shape, mode=lib.DFT3D_KDFT, flags=sf)
    y = fft(x)
    z = kdft(x)
    _finish(fft)
    kdft.status()
    ref = oracle.dft3d(x.cpu().numpy())
    assert oracle.rel_l2(y.cpu().numpy(), ref) < SANITY
    assert oracle.rel_l2(y.cpu().numpy(), z.cpu().numpy()) < TOL      # the two formulations agree
    assert torch.equal(x, _inputs().cube(shape, "uniform", 62, device="cuda"))  # input untouched
    inv = lib.Plan(*shape, mode=lib.DFT3D_FFT, sign=lib.DFT3D_INVERSE, flags=sf)
    back = inv(y)
    _finish(inv)
    assert oracle.rel_l2(back.cpu().numpy(), x.cpu().numpy()) < SANITY
    raw = lib.Plan(*shape, mode=lib.DFT3D_FFT, sign=lib.DFT3D_INVERSE, flags=lib.DFT3D_UNSCALED_INVERSE | sf)
    w = raw(y)
    _finish(raw)
    assert oracle.rel_l2(w.cpu().numpy() / np.prod(shape), x.cpu().numpy()) < SANITY
    for p in (fft, kdft, inv, raw):
        p.destroy()


@pytest.mark.parametrize("split", SPLITS)
@pytest.mark.parametrize("shape", [(256, 512, 256), (1024, 256, 256), (512, 1024, 256), (256, 4096, 256),
                                   (2048, 2048, 256)])
def test_fft_schedules_agree(lib, oracle, split, shape):
    """With a cube of workspace the 3D FFT goes in -> out (blocked order) -> workspace -> out; without it the
    three passes run in place on out.  The small shape: both against the oracle.  The longer ones (1024-point strided
    axes, the blocked layout with 16-line and 8-line stages): against each other and against the KDFT kernels, whose
    single axes are checked against the oracle above.  (2048, 2048, 256): both strided passes have 8-line stages, where
    the fp16 kernel interleaves pairs of rows in the blocked order so that the axis-1 pass reads whole 128-byte lines."""
    sf = _split_flag(lib, split)
    if max(shape) == 4096 and split == "tf32":
        pytest.skip("4096-point axes exist with fp16 pieces only")
    x = _inputs().cube(shape, "normal", 66, device="cuda")
    with_ws = lib.Plan(*shape, mode=lib.DFT3D_FFT, flags=sf)
    in_place = lib.Plan(*shape, mode=lib.DFT3D_FFT, workspace_limit=1 << 20, flags=sf)
    assert in_place.workspace_bytes == 0
    if shape != (256, 512, 256):
        # (a plan skips the workspace when the stage widths of its axis-0 and axis-1 passes do not nest)
        a, b = with_ws(x), in_place(x)
        _finish(with_ws)
        in_place.status()
        kd = lib.Plan(*shape, mode=lib.DFT3D_KDFT)
        c = kd(x)
        _finish(kd)
        assert _rel_l2_gpu(a, b) < SANITY and _rel_l2_gpu(a, c) < TOL
        for plan in (with_ws, in_place, kd):
            plan.destroy()
        return
    ref = oracle.dft3d(x.cpu().numpy())
    assert with_ws.workspace_bytes == x.numel() * 8
    for plan in (with_ws, in_place):
        y = plan(x)
        _finish(plan)
        assert oracle.rel_l2(y.cpu().numpy(), ref) < SANITY
        plan.destroy()


@pytest.mark.parametrize("shape", [(256, 256, 512), (2048, 2048, 256), (256, 4096, 256)])
def test_fft_half_cube_workspace(lib, oracle, shape):
    """When a whole cube of workspace is too much but a half (quarter, eighth) is not, the two strided passes run once
    per half (quarter, eighth) of the last axis (slice of the natural input -> blocked order in the workspace -> that half of `out` in natural
    order) and the contiguous pass runs in place on `out`: five launches.  The small shape against the oracle; the
    others (8-line stages with interleaved rows; 16-line axis-0 blocks read by 4-line axis-1 stages) against the
    in-place schedule."""
    x = _inputs().cube(shape, "normal", 68, device="cuda")
    half_bytes = x.numel() * 8 // 2
    half = lib.Plan(*shape, mode=lib.DFT3D_FFT, workspace_limit=half_bytes)
    assert half.workspace_bytes == half_bytes and half.launches == 5
    a = half(x)
    _finish(half)
    half.destroy()
    # an eighth of a cube: eight slices, seventeen launches, the same result as with two slices up to rounding order
    # (bit for bit in fact: the slices only regroup independent columns)
    eighth = lib.Plan(*shape, mode=lib.DFT3D_FFT, workspace_limit=half_bytes // 4)
    assert eighth.workspace_bytes == half_bytes // 4 and eighth.launches == 17
    a8 = eighth(x)
    _finish(eighth)
    eighth.destroy()
    assert torch.equal(a, a8)
    del a8
    if shape == (256, 256, 512):
        assert oracle.rel_l2(a.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
        inv = lib.Plan(*shape, mode=lib.DFT3D_FFT, sign=lib.DFT3D_INVERSE, workspace_limit=half_bytes // 2)
        assert inv.launches == 9
        back = inv(a)
        _finish(inv)
        inv.destroy()
        assert _rel_l2_gpu(back, x) < SANITY
        return
    in_place = lib.Plan(*shape, mode=lib.DFT3D_FFT, workspace_limit=1 << 20)
    assert in_place.workspace_bytes == 0 and in_place.launches == 3
    b = in_place(x)
    _finish(in_place)
    in_place.destroy()
    assert _rel_l2_gpu(a, b) < SANITY


@pytest.mark.parametrize("shape", [(256, 256, 256), pytest.param((256, 1024, 1024), marks=pytest.mark.slow),
                                   (512, 1024, 1024), (1024, 256, 256)])
def test_fft_two_axes_in_one_launch(lib, oracle, shape, monkeypatch):
    """With DFT3D_FFT_FUSE=1, plans whose axes 1 and 2 have the same length R*R run those two axes in ONE launch: the
    CTAs of the axis-1 pass hand n0-planes to the CTAs of the axis-2 pass through a small ring (two launches per
    transform instead of three).  The arithmetic of every line is that of the one-axis kernels, so the result equals
    the three-launch schedule bit for bit; the first two shapes also go against the full float64 oracle."""
    x = _inputs().cube(shape, "normal", 70, device="cuda")
    plain = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    assert plain.launches == 3
    monkeypatch.setenv("DFT3D_FFT_FUSE", "1")
    fused = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    assert fused.launches == 2
    a = fused(x)
    _finish(fused)
    b = plain(x)
    _finish(plain)
    plain.destroy()
    assert torch.equal(a, b)
    del b
    # again, with the ring and its counters left over from the first run, and with a very short ring
    a2 = fused(x)
    _finish(fused)
    fused.destroy()
    assert torch.equal(a, a2)
    monkeypatch.setenv("DFT3D_FFT_FUSE_RING", "2")
    monkeypatch.setenv("DFT3D_FFT_FUSE_WRITERS", "37")
    monkeypatch.setenv("DFT3D_FFT_FUSE_HINTS", "1")
    short = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    monkeypatch.delenv("DFT3D_FFT_FUSE_RING")
    monkeypatch.delenv("DFT3D_FFT_FUSE_WRITERS")
    monkeypatch.delenv("DFT3D_FFT_FUSE_HINTS")
    a2 = short(x)
    _finish(short)
    short.destroy()
    assert torch.equal(a, a2)
    del a2
    if shape[1] * shape[2] * shape[0] <= 256 * 1024 * 1024 and shape[0] == 256:
        assert oracle.rel_l2(a.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
    inv = lib.Plan(*shape, mode=lib.DFT3D_FFT, sign=lib.DFT3D_INVERSE)
    monkeypatch.delenv("DFT3D_FFT_FUSE")
    assert inv.launches == 2
    back = inv(a)
    _finish(inv)
    inv.destroy()
    assert _rel_l2_gpu(back, x) < SANITY


@pytest.mark.slow
def test_fft_blocked_order_with_four_rows_per_line(lib):
    """4096-point strided axes have 4-line stages (32-byte pieces): in the blocked order between the axis-0 and the
    axis-1 pass four neighbouring rows share each 128-byte line.  Needs 4096 points on axes 0 AND 1, i.e. 32 GiB per
    cube; compared with the in-place schedule (whose 4096-point passes are checked against the oracle axis by axis)."""
    free, total = torch.cuda.mem_get_info()
    if total < 170 * 2 ** 30:
        pytest.skip("needs a 180 GB device")
    shape = (4096, 4096, 256)
    x = _inputs().cube(shape, "normal", 67, device="cuda")
    with_ws = lib.Plan(*shape, mode=lib.DFT3D_FFT, workspace_limit=40 * 2 ** 30)
    assert with_ws.workspace_bytes == x.numel() * 8
    a = with_ws(x)
    _finish(with_ws)
    with_ws.destroy()
    in_place = lib.Plan(*shape, mode=lib.DFT3D_FFT, workspace_limit=1 << 20)
    assert in_place.workspace_bytes == 0
    b = in_place(x)
    _finish(in_place)
    in_place.destroy()
    assert _rel_l2_gpu(a, b) < SANITY


@pytest.mark.parametrize("mode", ["kdft", "fft"])
def test_execute_is_capturable_in_a_cuda_graph(lib, mode):
    """dft3d_execute only enqueues work on the stream (no allocation, no synchronisation, no host-side reads of device
    state), so a transform can be captured into a CUDA graph and replayed on new data in the same buffers."""
    shape = (64, 128, 256) if mode == "kdft" else (256, 256, 256)
    plan = lib.Plan(*shape, mode=lib.DFT3D_KDFT if mode == "kdft" else lib.DFT3D_FFT)
    x = _inputs().cube(shape, "normal", 410, device="cuda")
    y = torch.empty_like(x)
    plan(x, y)                      # eager, also the warm-up
    _finish(plan)
    want = y.clone()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    y.zero_()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            plan.execute(x, y, stream=side)
    graph.replay()
    _finish(plan)
    assert torch.equal(y, want)
    x2 = _inputs().cube(shape, "normal", 411, device="cuda")
    x.copy_(x2)
    graph.replay()
    _finish(plan)
    got = y.clone()
    plan(x2, y)
    _finish(plan)
    assert torch.equal(got, y)
    plan.destroy()


def test_execute_host_batch_matches_single_calls(lib, oracle):
    """The streamed host entry point (two device buffer pairs, uploads and downloads on their own streams) gives,
    cube by cube, the bits of dft3d_execute_host; five cubes so that both buffer pairs are reused; one against the
    oracle.  A plan that uses its input buffer as workspace must not lose an upload to the previous transform."""
    shape = (64, 128, 256)
    xs = [_inputs().cube(shape, "normal", 300 + i, device="cpu").pin_memory() for i in range(5)]
    for flags in (0, lib.DFT3D_DESTROY_INPUT):
        plan = lib.Plan(*shape, mode=lib.DFT3D_KDFT, flags=flags)
        want = []
        for x in xs:
            y = torch.empty_like(x).pin_memory()
            plan.execute_host(x, y)
            want.append(y)
        got = [torch.empty_like(x).pin_memory() for x in xs]
        plan.execute_host_batch(xs, got)
        for w, g in zip(want, got):
            assert torch.equal(w, g)
        plan.execute_host_batch([], [])
        one = [torch.empty_like(xs[0]).pin_memory()]
        plan.execute_host_batch(xs[:1], one)
        assert torch.equal(one[0], want[0])
        plan.destroy()
    assert oracle.rel_l2(got[3].numpy(), oracle.dft3d(xs[3].numpy())) < SANITY
    plan = lib.Plan(*shape, mode=lib.DFT3D_KDFT)
    with pytest.raises(ValueError):
        plan.execute_host_batch(xs, got[:2])
    plan.destroy()


@pytest.mark.parametrize("split", SPLITS)
def test_fft_mixed_axis_lengths(lib, oracle, split):
    shape = (256, 1024, 256)
    x = _inputs().cube(shape, "normal", 63, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, fft_split=((16, 16), (32, 32), None), flags=_split_flag(lib, split))
    y = plan(x)
    _finish(plan)
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
    plan.destroy()
    with pytest.raises(lib.Dft3dError) as e:
        lib.Plan(*shape, mode=lib.DFT3D_FFT, fft_split=((32, 8), None, None))
    assert e.value.status == 2
    with pytest.raises(lib.Dft3dError) as e:
        lib.Plan(768, 256, 256, mode=lib.DFT3D_FFT)
    assert e.value.status == 2


@pytest.mark.parametrize("shape,axis", [((256, 256, 512), 2), ((256, 512, 256), 1), ((512, 256, 256), 0),
                                        ((256, 256, 2048), 2), ((256, 2048, 256), 1), ((2048, 256, 256), 0),
                                        ((256, 256, 4096), 2), ((256, 4096, 256), 1), ((4096, 256, 256), 0)])
@pytest.mark.parametrize("split", SPLITS)
def test_fft_radix2_lengths_single_axis(lib, oracle, shape, axis, split):
    """N = 2*R*R (512 = 2*16*16, 2048 = 2*32*32) and N = 4*R*R (4096 = 4*32*32, fp16 pieces only): butterfly + two
    GEMM stages.  The oracle transforms a slab of 8 lines-worth along an untransformed axis (lines are independent),
    which keeps the long cases short."""
    if max(shape) == 4096 and split == "tf32":
        with pytest.raises(lib.Dft3dError) as e:
            lib.Plan(*shape, mode=lib.DFT3D_FFT, flags=_split_flag(lib, split))
        assert e.value.status == 2
        return
    x = _inputs().cube(shape, "normal", 64 + axis, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, flags=_split_flag(lib, split))
    y = plan.execute_axis(axis, x)
    _finish(plan)
    plan.destroy()
    sl = (slice(None), slice(0, 8), slice(None)) if axis == 0 else (slice(0, 8), slice(None), slice(None))
    ref = oracle.dft_axis(x[sl].cpu().numpy().astype(np.complex128), axis)
    err = oracle.rel_l2(y[sl].cpu().numpy(), ref)
    assert err < SANITY_AXIS, (shape, axis, err)
    # the rest of the output against the (oracle-checked) KDFT kernel of the same axis
    kdft = lib.Plan(*shape, mode=lib.DFT3D_KDFT)
    z = kdft.execute_axis(axis, x)
    _finish(kdft)
    kdft.destroy()
    assert _rel_l2_gpu(y, z) < TOL


def test_fft_512_cube_forward_inverse(lib, oracle):
    shape = (512, 256, 512)
    x = _inputs().cube(shape, "uniform", 65, device="cuda")
    fwd = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    inv = lib.Plan(*shape, mode=lib.DFT3D_FFT, sign=lib.DFT3D_INVERSE)
    y = fwd(x)
    back = inv(y)
    _finish(inv)
    fwd.status()
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
    assert oracle.rel_l2(back.cpu().numpy(), x.cpu().numpy()) < SANITY
    fwd.destroy()
    inv.destroy()


# ------------------------------------------------------------------ config 3: 1024^3, FFT (32*32) against KDFT and the oracle

def _rel_l2_gpu(a, b):
    """||a - b|| / ||b|| over complex values, accumulated in float64 on the device plane by plane."""
    num = torch.zeros((), dtype=torch.float64, device=a.device)
    den = torch.zeros((), dtype=torch.float64, device=a.device)
    for i in range(a.shape[0]):
        d = (a[i].to(torch.complex128) - b[i].to(torch.complex128))
        num += (d.real ** 2 + d.imag ** 2).sum()
        bb = b[i].to(torch.complex128)
        den += (bb.real ** 2 + bb.imag ** 2).sum()
    return float(torch.sqrt(num / den))


@pytest.mark.slow
def test_config3_fft_1024_vs_kdft_and_oracle_subset(lib, oracle):
    n = 1024
    shape = (n, n, n)
    inp = _inputs()
    x = inp.cube(shape, "uniform", 1003, device="cuda")
    fft = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    y = fft(x)
    _finish(fft)
    fft.destroy()
    kdft = lib.Plan(*shape, mode=lib.DFT3D_KDFT)
    z = kdft(x)
    _finish(kdft)
    kdft.destroy()
    assert _rel_l2_gpu(y, z) < TOL                     # full-array agreement of the two formulations
    # Parseval on the full output (uniform grid): sum |X|^2 = P sum |x|^2
    ex = sum(float((torch.view_as_real(x[i]).double() ** 2).sum()) for i in range(n))
    ey = sum(float((torch.view_as_real(y[i]).double() ** 2).sum()) for i in range(n))
    assert abs(ey / (float(n) ** 3 * ex) - 1.0) < 1e-5
    # 18^3 coefficients on a stratified product grid by the float64 oracle (each its full triple sum)
    S = [inp.stratified_indices(n, 16, 3003 + a) for a in range(3)]
    sub = oracle.Subset(shape, S[0], S[1], S[2])
    for a in range(0, n, 64):
        sub.feed(x[a:a + 64].cpu().numpy())
    ref = sub.result()
    ix = np.ix_(S[0], S[1], S[2])
    idx = [torch.as_tensor(s, device="cuda") for s in S]
    got_fft = y[idx[0]][:, idx[1]][:, :, idx[2]].cpu().numpy()
    got_kdft = z[idx[0]][:, idx[1]][:, :, idx[2]].cpu().numpy()
    assert ref.shape == got_fft.shape and ref.size >= 4096
    assert oracle.rel_l2(got_fft, ref) < TOL
    assert oracle.rel_l2(got_kdft, ref) < TOL
    # two coefficients by the literal triple loop: the evaluator with shared partial sums hides nothing, and the
    # GPU value is close to it.  The per-coefficient bound is looser than the norm-wise one: at k = (0,0,0) the
    # tiny systematic part of the rounding errors of all 2^30 samples adds up coherently.
    xh = x.cpu().numpy()
    rms = np.sqrt(float(n) ** 3 * 2.0 / 3.0)              # rms coefficient magnitude for U(-1,1) input
    for pos in ((0, 0, 0), (3, 5, 7)):
        k = tuple(int(S[a][pos[a]]) for a in range(3))
        want = oracle.coeff_triple(xh, k)
        assert abs(want - ref[pos]) < 1e-9 * rms, (k, want, ref[pos])
        got = complex(y[k].item())
        assert abs(got - want) < 5e-5 * rms, (k, got, want, abs(got - want) / rms)


# ------------------------------------------------------------------ config 5: 2048^3 (64 GiB in, 64 GiB out), both formulations

@pytest.mark.slow
def test_config5_2048_exponentials_both_modes(lib, oracle):
    """Largest single-GPU instance.  Input: 16 unit exponentials (distinct integer frequencies, seeded phases)
    plus N(0, sigma = 1e-3) noise, so the spectrum is 16 peaks of magnitude P over a floor of about sigma*sqrt(2P).
    Only two 64 GiB tensors (and a fraction of a cube of workspace) fit, so FFT and KDFT run one after the other into the same output and are compared
    on sampled planes; each is compared with the float64 oracle on a product grid of coefficients that contains
    all peaks.  Gate: the norm-wise relative L2 error of the whole output, estimated from the subset by strata.
    A coefficient's error level depends on how many of its three indices coincide with a peak's index on that axis
    (it then lies on a line or plane that carried a peak through one or two of the axis passes), and the product
    grid over-represents those; so the samples are grouped by that count c = 0..3, each group's mean |d|^2 is scaled
    to the group's true population N_c, and rel^2 = sum_c N_c * mean_c |d|^2 / (P * sum|x|^2) <= 1e-10 (the
    denominator is the output energy by Parseval).  Also: every peak within 1e-5 relative, Parseval to 1e-5.
    """
    free, total = torch.cuda.mem_get_info()
    if total < 170 * 2 ** 30:
        pytest.skip("needs a 180 GB device")
    n = 2048
    shape = (n, n, n)
    P = float(n) ** 3
    inp = _inputs()
    x, freqs, phases = inp.exponentials(shape, 16, 2005, 1e-3, 1005, device="cuda")
    ex = sum(float((torch.view_as_real(x[i]).double() ** 2).sum()) for i in range(n))
    S = [inp.stratified_indices(n, 16, 5005 + a, forced=freqs[:, a]) for a in range(3)]
    sub = oracle.Subset(shape, S[0], S[1], S[2])
    for a in range(0, n, 32):
        sub.feed(x[a:a + 32].cpu().numpy())
    ref = sub.result()
    pos = [{int(v): i for i, v in enumerate(S[a])} for a in range(3)]
    peak_pos = [tuple(pos[a][int(f[a])] for a in range(3)) for f in freqs]
    # closed form of the peaks: P * exp(i phi) up to the noise term (a few sigma*sqrt(2P) = 130)
    for e, pp in enumerate(peak_pos):
        assert abs(ref[pp] - P * np.exp(1j * phases[e])) < 2000.0
    # strata: number of axes on which the sample's index is some peak's index; exact population of each stratum
    F = [np.unique(freqs[:, a]) for a in range(3)]
    on = [np.isin(S[a], F[a]) for a in range(3)]
    count = on[0][:, None, None].astype(int) + on[1][None, :, None] + on[2][None, None, :]
    u = [len(f) for f in F]
    pop = [float((n - u[0]) * (n - u[1]) * (n - u[2])),
           float(u[0] * (n - u[1]) * (n - u[2]) + (n - u[0]) * u[1] * (n - u[2]) + (n - u[0]) * (n - u[1]) * u[2]),
           float(u[0] * u[1] * (n - u[2]) + u[0] * (n - u[1]) * u[2] + (n - u[0]) * u[1] * u[2]),
           float(u[0] * u[1] * u[2])]
    assert abs(sum(pop) - P) < 1.0 and all((count == c).sum() > 0 for c in range(4))
    assert (count == 3).sum() == pop[3]          # the grid holds every point of the innermost stratum
    idx = [torch.as_tensor(s, device="cuda") for s in S]
    planes = [torch.as_tensor(inp.stratified_indices(n, 16, 6005 + a), device="cuda") for a in range(3)]
    out = torch.empty_like(x)
    kept = None
    floor_only = {}
    for mode, split in ((lib.DFT3D_FFT, "fp16"), (lib.DFT3D_KDFT, "fp16"), (lib.DFT3D_FFT, "tf32")):
        # FFT: the default limit (16 GiB), i.e. a quarter of a cube of workspace beside the two cubes and the strided
        # passes once per quarter of the last axis; KDFT: groups of planes.  The TF32-piece FFT plan (three passes in
        # place) is there for the floor-only figure below.
        sf = _split_flag(lib, split)
        plan = lib.Plan(*shape, mode=mode, flags=sf) if mode == lib.DFT3D_FFT else lib.Plan(*shape, mode=mode, workspace_limit=4 * 2 ** 30, flags=sf)
        if mode == lib.DFT3D_FFT and split == "fp16":
            assert plan.workspace_bytes == x.numel() * 2 and plan.launches == 9
        plan(x, out)
        _finish(plan)
        plan.destroy()
        got = out[idx[0]][:, idx[1]][:, :, idx[2]].cpu().numpy()
        d2 = np.abs(got - ref) ** 2
        strata = [pop[c] * d2[count == c].mean() for c in range(4)]
        est = sum(strata) / (P * ex)
        assert est < TOL ** 2, (mode, np.sqrt(est), [np.sqrt(v / (P * ex)) for v in strata])
        # Reported, not gated: the error of the floor-only coefficients (no index shared with a peak) normalised by
        # their OWN norm.  No fp32 pipeline can bring this to 1e-5: a floor coefficient is what is left after
        # peak-sized terms cancel, and it inherits their rounding.
        name = ("fft" if mode == lib.DFT3D_FFT else "kdft") + "_" + split
        floor_only[name] = float(np.sqrt(d2[count == 0].sum() / (np.abs(ref[count == 0]) ** 2).sum()))
        print("config 5, %s: norm-wise estimate %.3g, floor-only subset-normalised error %.3g"
              % (name, np.sqrt(est), floor_only[name]))
        if split == "tf32":
            continue
        for pp in peak_pos:
            assert abs(got[pp] - ref[pp]) < TOL * abs(ref[pp]), (mode, pp, got[pp], ref[pp])
        ey = sum(float((torch.view_as_real(out[i]).double() ** 2).sum()) for i in range(n))
        assert abs(ey / (P * ex) - 1.0) < TOL, (mode, ey / (P * ex))
        sampled = [out[planes[0]].clone(), out[:, planes[1]].clone(), out[:, :, planes[2]].clone()]
        if kept is None:
            kept = sampled
        else:
            for a, b in zip(sampled, kept):      # KDFT against FFT on planes that cross every output tile
                num = float(((a.to(torch.complex128) - b.to(torch.complex128)).abs() ** 2).sum())
                den = float((b.to(torch.complex128).abs() ** 2).sum())
                # planes that miss the peaks hold only the noise floor, which fp32 accumulation cannot resolve to
                # 1e-5 of itself; the error is measured against the mean |X|^2 of the full spectrum, which by
                # Parseval is sum|x|^2
                assert num / a.numel() < (TOL ** 2) * ex, (num / a.numel(), den / a.numel(), ex)
    del kept
    import json
    import os
    record = os.environ.get("DFT3D_RECORD_DIR")          # where to keep the reported (not gated) figures, if anywhere
    if record and os.path.isdir(record):
        with open(os.path.join(record, "config5_floor_only_error.json"), "w") as f:
            json.dump(floor_only, f)


# ------------------------------------------------------------------ batched 2D / 1D transforms (subset of the axes)

def _oracle_axes(oracle, xh, axes, **kw):
    y = xh.astype(np.complex128)
    for a in axes:
        y = oracle.dft_axis(y, a, **kw)
    return y


@pytest.mark.parametrize("mode_name,shape", [("kdft", (3, 128, 192)), ("kdft", (1, 64, 256)), ("fft", (5, 256, 512))])
def test_batched_2d(lib, oracle, mode_name, shape):
    """axes=(1,2): n0 independent 2D transforms X = V1 x V2^T (Eq. 5); n0 need not be a multiple of 64."""
    mode = lib.DFT3D_KDFT if mode_name == "kdft" else lib.DFT3D_FFT
    x = _inputs().cube(shape, "normal", 81, device="cuda")
    plan = lib.Plan(*shape, mode=mode, axes=(1, 2))
    y = plan(x)
    _finish(plan)
    assert plan.launches == _pre(lib, plan, mode_name == "kdft") + 2
    plan.destroy()
    err = oracle.rel_l2(y.cpu().numpy(), _oracle_axes(oracle, x.cpu().numpy(), (1, 2)))
    assert err < SANITY, (mode_name, shape, err)


@pytest.mark.parametrize("axes", [(2,), (1,), (0,), (0, 1), (0, 2)])
@pytest.mark.parametrize("split", SPLITS)
def test_axis_subsets_kdft(lib, oracle, axes, split):
    shape = (64, 128, 64)
    x = _inputs().cube(shape, "uniform", 82, device="cuda")
    plan = lib.Plan(*shape, axes=axes, sign=lib.DFT3D_INVERSE, flags=_split_flag(lib, split))
    y = plan(x)
    _finish(plan)
    assert plan.launches == _pre(lib, plan) + len(axes)
    with pytest.raises(lib.Dft3dError):
        plan.execute_axis([a for a in range(3) if a not in axes][0], x)
    plan.destroy()
    ref = x.cpu().numpy().astype(np.complex128)
    for a in axes:
        ref = oracle.dft_axis(ref, a, sign=+1, scale=1.0 / shape[a])
    assert oracle.rel_l2(y.cpu().numpy(), ref) < SANITY, axes


def test_batched_1d_fft(lib, oracle):
    shape = (7, 64, 1024)
    x = _inputs().cube(shape, "normal", 83, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, axes=(2,))
    y = plan(x)
    _finish(plan)
    plan.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), _oracle_axes(oracle, x.cpu().numpy(), (2,))) < SANITY_AXIS


# ------------------------------------------------------------------ sizes that are not tile multiples (KDFT)

@pytest.mark.parametrize("shape", [(100, 66, 250), (30, 18, 34), (2, 4, 6), (130, 64, 2), (66, 258, 64),
                                   (100, 68, 36), (4, 132, 252), (260, 8, 12),
                                   (3, 5, 6), (129, 33, 64), (1, 7, 2), (5, 64, 130), (255, 1, 8)])
def test_kdft_general_even_sizes(lib, oracle, shape):
    """Any length on axes 0 and 1, any even length on the last axis: ragged K stages are zero-filled by TMA on both
    operands, ragged tiles masked on store, and an odd length pads the rows of the TABLE to a 16-byte multiple (the
    data is never padded).  Shapes whose lengths are all multiples of 4 run the fp16 split, the others the TF32 split."""
    x = _inputs().cube(shape, "normal", 91, device="cuda")
    guard = torch.full((1 << 14,), 7.0, device="cuda")           # canaries around the output
    out = torch.empty_like(x)
    guard2 = torch.full((1 << 14,), 7.0, device="cuda")
    plan = lib.Plan(*shape)
    fp16_ok = all(n % 4 == 0 for n in shape)
    assert plan.split == (lib.DFT3D_SPLIT_FP16 if fp16_ok else lib.DFT3D_SPLIT_TF32)
    if not fp16_ok:
        with pytest.raises(lib.Dft3dError):
            lib.Plan(*shape, flags=lib.DFT3D_SPLIT_FP16)
    plan(x, out)
    _finish(plan)
    plan.destroy()
    err = oracle.rel_l2(out.cpu().numpy(), oracle.dft3d(x.cpu().numpy()))
    assert err < SANITY, (shape, err)
    assert bool((guard == 7.0).all()) and bool((guard2 == 7.0).all())
    nodes = _inputs().sorted_nodes(shape, 92)
    plan = lib.Plan(*shape, nodes=nodes)
    y = plan(x)
    _finish(plan)
    plan.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy(), nodes=nodes)) < SANITY


def test_kdft_refuses_an_odd_last_axis(lib):
    """Rows of the data are 8*n2 bytes long and TMA needs them to start on 16-byte boundaries: an odd last axis is
    refused with a message that says so, whether or not that axis is transformed."""
    for axes in (None, (0, 1)):
        with pytest.raises(lib.Dft3dError) as e:
            lib.Plan(8, 6, 7, axes=axes)
        assert e.value.status == 2 and "16-byte" in str(e.value)


# ------------------------------------------------------------------ fp16 split: scaling by powers of two

@pytest.mark.parametrize("log2_scale", [-120, -60, 0, 90])
def test_fp16_split_is_scale_invariant(lib, oracle, log2_scale):
    """The fp16 pieces are taken after an exact power-of-two scaling chosen from the largest input magnitude, so
    a scaled input gives the scaled result bit for bit (2^-120 puts the data next to the smallest normal float,
    where the scale factor saturates and a few entries are subnormal: fp32-level accuracy is all that is asked)."""
    shape = (64, 128, 64)
    x = _inputs().cube(shape, "normal", 93, device="cuda")
    plan = lib.Plan(*shape, flags=lib.DFT3D_SPLIT_FP16)
    y = plan(x).clone()
    xs = x * (2.0 ** log2_scale)
    ys = plan(xs)
    _finish(plan)
    plan.destroy()
    if log2_scale > -100:
        assert torch.equal(ys, y * (2.0 ** log2_scale))
    ref = oracle.dft3d(xs.cpu().numpy().astype(np.complex128))
    assert oracle.rel_l2(ys.cpu().numpy().astype(np.complex128), ref) < SANITY


def test_fp16_split_wide_dynamic_range(lib, oracle):
    """One entry 2^30 above the rest: the error stays at fp32 level relative to the norm of the result (small
    entries lose relative, not norm-wise, accuracy), and the TF32 split agrees."""
    shape = (64, 64, 128)
    x = _inputs().cube(shape, "normal", 94, device="cuda")
    x[3, 5, 7] = 2.0 ** 30
    ref = oracle.dft3d(x.cpu().numpy())
    for flag in (lib.DFT3D_SPLIT_FP16, lib.DFT3D_SPLIT_TF32):
        plan = lib.Plan(*shape, flags=flag)
        y = plan(x)
        _finish(plan)
        plan.destroy()
        assert oracle.rel_l2(y.cpu().numpy(), ref) < SANITY, flag
    # all-zero input: no scale is derived, the result is exactly zero
    plan = lib.Plan(*shape, flags=lib.DFT3D_SPLIT_FP16)
    z = plan(torch.zeros_like(x))
    _finish(plan)
    plan.destroy()
    assert not bool(z.any())


@pytest.mark.slow
def test_splits_agree_512(lib, oracle):
    """Config-2 size: the two splits agree with each other to fp32 level and the fp16 one is not slower."""
    shape = (512, 512, 512)
    x = _inputs().cube(shape, "uniform", 95, device="cuda")
    res = {}
    for name in SPLITS:
        plan = lib.Plan(*shape, flags=_split_flag(lib, name))
        res[name] = plan(x)
        _finish(plan)
        plan.destroy()
    diff = torch.linalg.vector_norm((res["fp16"] - res["tf32"]).flatten()) / torch.linalg.vector_norm(res["tf32"].flatten())
    assert diff.item() < SANITY


@pytest.mark.parametrize("axis", [1, 2])
@pytest.mark.parametrize("shape", [(64, 256, 256), (64, 512, 512)])     # 256 = 16*16; 512 = 2*16*16 (radix-2 step first)
def test_fft_fp16_scales_every_line_on_its_own(lib, oracle, axis, shape):
    """The fp16 split of the FFT kernel scales each line by a power of two taken from that line's largest element.
    Lines that differ by up to 2^120 in magnitude must each come out with fp32-level error relative to their OWN norm
    (a single scale for the whole array would flush the small lines to zero)."""
    x = _inputs().cube(shape, "normal", 96, device="cuda")
    g = torch.Generator(device="cuda").manual_seed(97)
    other = [d for d in range(3) if d != axis]
    expo = torch.randint(-60, 61, [shape[d] for d in other], generator=g, device="cuda").to(torch.float32)
    scale = torch.exp2(expo).unsqueeze(axis)
    xs = (x * scale).contiguous()
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, flags=lib.DFT3D_SPLIT_FP16, axes=(axis,))
    ys = plan(xs)
    _finish(plan)
    plan.destroy()
    assert bool(torch.isfinite(torch.view_as_real(ys)).all())
    ref = oracle.dft_axis(x.cpu().numpy().astype(np.complex128), axis)     # unscaled lines: scaling by 2^k is exact
    got = (ys / scale).cpu().numpy().astype(np.complex128)
    err = np.sqrt((np.abs(got - ref) ** 2).sum(axis=axis) / (np.abs(ref) ** 2).sum(axis=axis))
    assert err.max() < SANITY_AXIS, err.max()


@pytest.mark.parametrize("mode_name,shape", [("kdft", (64, 128, 192)), ("fft", (256, 512, 256)), ("fft", (1024, 256, 256))])
def test_destroy_input_uses_the_input_as_workspace(lib, oracle, mode_name, shape):
    """DFT3D_DESTROY_INPUT: no workspace is allocated, the input cube is overwritten, the result is the same."""
    mode = lib.DFT3D_KDFT if mode_name == "kdft" else lib.DFT3D_FFT
    x = _inputs().cube(shape, "normal", 98, device="cuda")
    keep = lib.Plan(*shape, mode=mode)
    want = keep(x)
    _finish(keep)
    keep.destroy()
    plan = lib.Plan(*shape, mode=mode, flags=lib.DFT3D_DESTROY_INPUT)
    assert plan.workspace_bytes == 0
    scratch = x.clone()
    got = plan(scratch)
    _finish(plan)
    plan.destroy()
    assert _rel_l2_gpu(got, want) < SANITY
    if shape[0] <= 256:
        assert oracle.rel_l2(got.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
    assert not torch.equal(scratch, x)      # the input really served as scratch


def test_kdft_cta_pair_kernel_matches(lib, oracle, monkeypatch):
    """The cta_group::2 form of the fp16 KDFT kernel (pairs of CTAs share every table tile; enabled with
    DFT3D_KDFT_PAIR=1 at plan creation) computes the same sums in the same order: identical bits, and a ragged
    shape against the oracle."""
    shape = (256, 128, 384)
    x = _inputs().cube(shape, "normal", 99, device="cuda")
    plan = lib.Plan(*shape, flags=lib.DFT3D_SPLIT_FP16)
    want = plan(x)
    _finish(plan)
    plan.destroy()
    monkeypatch.setenv("DFT3D_KDFT_PAIR", "1")
    plan = lib.Plan(*shape, flags=lib.DFT3D_SPLIT_FP16)
    got = plan(x)
    _finish(plan)
    plan.destroy()
    assert torch.equal(got, want)
    shape = (132, 260, 200)
    x = _inputs().cube(shape, "normal", 100, device="cuda")
    plan = lib.Plan(*shape, flags=lib.DFT3D_SPLIT_FP16)
    y = plan(x)
    _finish(plan)
    plan.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY


# ------------------------------------------------------------------ the largest supported length

@pytest.mark.parametrize("axis", [0, 2])
def test_kdft_maximum_length_8192(lib, oracle, axis):
    """n_a = 8192 is the longest axis the KDFT kernels take (table: 2 x 16384^2 fp16 = 1 GiB); a thin slab keeps the
    oracle cheap."""
    shape = (8192, 4, 2) if axis == 0 else (2, 4, 8192)
    x = _inputs().cube(shape, "normal", 101, device="cuda")
    plan = lib.Plan(*shape, axes=(axis,))
    y = plan(x)
    _finish(plan)
    plan.destroy()
    ref = oracle.dft_axis(x.cpu().numpy().astype(np.complex128), axis)
    assert oracle.rel_l2(y.cpu().numpy(), ref) < SANITY_AXIS
    with pytest.raises(lib.Dft3dError) as e:
        lib.Plan(2, 4, 8194, axes=(2,))
    assert e.value.status == 2


@pytest.mark.slow
def test_2d_kdft_8192_squared_separable_input(lib, oracle):
    """The paper's 2D workload (Section V-A: 2D KDFT of 8192 x 8192, Eq. 5 X = V1 x V2^T).  The full oracle would take
    minutes, so the input is a sum of three outer products a_i b_i^T, whose transform is the sum of the outer products
    of the 1D transforms (two 8192-point oracle transforms per term)."""
    n = 8192
    rng = np.random.default_rng(102)
    a = (rng.standard_normal((3, n)) + 1j * rng.standard_normal((3, n)))
    b = (rng.standard_normal((3, n)) + 1j * rng.standard_normal((3, n)))
    x64 = np.einsum("ij,ik->jk", a, b)
    x = torch.from_numpy(x64.astype(np.complex64)).reshape(1, n, n).cuda()
    # the oracle sees exactly what the GPU sees only if the terms are formed from the rounded input: use linearity on
    # the complex64 input instead (rank <= 3 no longer holds exactly after rounding), i.e. check against
    # sum_i F(a_i) F(b_i)^T up to the input's own rounding error (6e-8 relative), well inside the bound below
    fa = np.stack([oracle.dft_axis(a[i].reshape(1, 1, n), 2).reshape(n) for i in range(3)])
    fb = np.stack([oracle.dft_axis(b[i].reshape(1, 1, n), 2).reshape(n) for i in range(3)])
    ref = np.einsum("ij,ik->jk", fa, fb)
    plan = lib.Plan(1, n, n, axes=(1, 2))
    y = plan(x)
    _finish(plan)
    plan.destroy()
    got = y.cpu().numpy().reshape(n, n).astype(np.complex128)
    err = np.linalg.norm(got - ref) / np.linalg.norm(ref)
    assert err < SANITY, err


@pytest.mark.parametrize("shape,axis", [((4, 64, 8192), 2), ((2, 8192, 64), 1), ((8192, 64, 64), 0)])
def test_fft_8192_point_axis(lib, oracle, shape, axis):
    """8192 = 1024 * 8 (Eq. 17 once more): the fused 1024-point kernel over the eight stride-8 sub-sequences, then the
    phase adjustment and the 8-point DFT in a second launch.  Each axis alone against the oracle, forward and scaled
    inverse (axis 0, where the oracle would need a minute per direction: against the KDFT kernel, whose 8192-point axis 0
    has its own oracle test); the plan reports the factor pair."""
    x = _inputs().cube(shape, "normal", 110 + axis, device="cuda")
    xh = x.cpu().numpy().astype(np.complex128)
    for sign in (lib.DFT3D_FORWARD, lib.DFT3D_INVERSE):
        plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, sign=sign, axes=(axis,))
        assert plan.launches == 2 and plan.fft_split(axis) == (1024, 8)
        y = plan(x)
        _finish(plan)
        ya = plan.execute_axis(axis, x)
        _finish(plan)
        plan.destroy()
        assert torch.equal(y, ya)
        if axis == 0:
            kd = lib.Plan(*shape, mode=lib.DFT3D_KDFT, sign=sign, axes=(axis,))
            z = kd(x)
            _finish(kd)
            kd.destroy()
            assert _rel_l2_gpu(y, z) < SANITY_AXIS, (axis, sign)
            continue
        want = oracle.dft_axis(xh, axis, sign=sign, scale=(1.0 / 8192 if sign > 0 else 1.0))
        assert oracle.rel_l2(y.cpu().numpy(), want) < SANITY_AXIS, (axis, sign)


@pytest.mark.slow
def test_2d_fft_8192_squared_matches_kdft_and_separable_input(lib, oracle):
    """The paper's 2D workload (Section V-A, 8192 x 8192) in the FFT formulation: four launches.  Against the sum of
    outer products of 1D oracle transforms (as the KDFT test above), against the KDFT plan, and AUTO picks it."""
    n = 8192
    rng = np.random.default_rng(112)
    a = (rng.standard_normal((3, n)) + 1j * rng.standard_normal((3, n)))
    b = (rng.standard_normal((3, n)) + 1j * rng.standard_normal((3, n)))
    x = torch.from_numpy(np.einsum("ij,ik->jk", a, b).astype(np.complex64)).reshape(1, n, n).cuda()
    fa = np.stack([oracle.dft_axis(a[i].reshape(1, 1, n), 2).reshape(n) for i in range(3)])
    fb = np.stack([oracle.dft_axis(b[i].reshape(1, 1, n), 2).reshape(n) for i in range(3)])
    ref = np.einsum("ij,ik->jk", fa, fb)
    plan = lib.Plan(1, n, n, mode=lib.DFT3D_FFT, axes=(1, 2))
    assert plan.launches == 4 and plan.workspace_bytes == x.numel() * 8
    y = plan(x)
    _finish(plan)
    plan.destroy()
    got = y.cpu().numpy().reshape(n, n).astype(np.complex128)
    assert np.linalg.norm(got - ref) / np.linalg.norm(ref) < SANITY
    kd = lib.Plan(1, n, n, axes=(1, 2))
    z = kd(x)
    _finish(kd)
    kd.destroy()
    assert _rel_l2_gpu(y, z) < SANITY
    auto = lib.Plan(1, n, n, mode=lib.DFT3D_AUTO, axes=(1, 2))
    assert auto.launches == 4
    w = auto(x)
    _finish(auto)
    auto.destroy()
    assert torch.equal(w, y)


def test_fft_8192_with_other_axes_and_destroy_input(lib, oracle):
    """An 8192-point axis beside a 256-point axis: three launches through the plan's own cube, against the oracle."""
    shape = (2, 256, 8192)
    x = _inputs().cube(shape, "uniform", 113, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_FFT, axes=(1, 2))
    assert plan.launches == 3
    y = plan(x)
    _finish(plan)
    plan.destroy()
    want = _oracle_axes(oracle, x.cpu().numpy(), (1, 2))
    assert oracle.rel_l2(y.cpu().numpy(), want) < SANITY
    with pytest.raises(lib.Dft3dError) as e:
        lib.Plan(*shape, mode=lib.DFT3D_FFT, axes=(1, 2), flags=lib.DFT3D_SPLIT_TF32)
    assert e.value.status == 2


@pytest.mark.slow
def test_fft_3d_with_an_8192_point_axis_and_the_input_as_workspace(lib):
    """A 3D plan with one 8192-point axis: four launches through the plan's cube, against the KDFT kernels (whose axes
    are checked against the oracle one by one).  With DFT3D_AUTO over an 8192-point axis 0 (two passes) and a 100-point
    axis 1 (KDFT) there are three passes, an odd number, so DFT3D_DESTROY_INPUT may use the input cube as the workspace."""
    shape = (256, 256, 8192)
    x = _inputs().cube(shape, "normal", 114, device="cuda")
    fft = lib.Plan(*shape, mode=lib.DFT3D_FFT)
    assert fft.launches == 4 and fft.workspace_bytes == x.numel() * 8
    a = fft(x)
    _finish(fft)
    fft.destroy()
    kd = lib.Plan(*shape, mode=lib.DFT3D_KDFT)
    b = kd(x)
    _finish(kd)
    kd.destroy()
    assert _rel_l2_gpu(a, b) < SANITY
    del a, b, x
    shape = (8192, 100, 128)
    x = _inputs().cube(shape, "normal", 115, device="cuda")
    auto = lib.Plan(*shape, mode=lib.DFT3D_AUTO, flags=lib.DFT3D_DESTROY_INPUT, axes=(0, 1))
    assert auto.workspace_bytes == 0 and auto.launches == 2 + 2     # two for the 8192-point axis, a reduction and a KDFT pass
    keep = lib.Plan(*shape, mode=lib.DFT3D_AUTO, axes=(0, 1))
    assert keep.workspace_bytes == x.numel() * 8
    want = keep(x)
    _finish(keep)
    keep.destroy()
    got = auto(x.clone())
    _finish(auto)
    auto.destroy()
    assert torch.equal(got, want)
    kd = lib.Plan(*shape, mode=lib.DFT3D_KDFT, axes=(0, 1))
    b = kd(x)
    _finish(kd)
    kd.destroy()
    assert _rel_l2_gpu(got, b) < SANITY


# ------------------------------------------------------------------ inverse nonuniform transform

@pytest.mark.parametrize("split", SPLITS)
def test_inverse_solve_undoes_the_nonuniform_forward_transform(lib, oracle, split):
    """DFT3D_INVERSE_SOLVE: nodes jittered around the uniform grid on two axes, a uniform third axis.  The solve
    plan returns the input of the forward plan, and agrees with the oracle's LAPACK solve of the same system."""
    shape = (64, 128, 192)
    rng = np.random.default_rng(103)
    nodes = [(np.arange(n) + 0.3 * rng.uniform(-1, 1, n)) / n for n in shape]
    nodes[1] = None
    x = _inputs().cube(shape, "normal", 104, device="cuda")
    sf = _split_flag(lib, split)
    fwd = lib.Plan(*shape, nodes=nodes, flags=sf)
    X = fwd(x)
    _finish(fwd)
    fwd.destroy()
    inv = lib.Plan(*shape, sign=lib.DFT3D_INVERSE, nodes=nodes, flags=sf | lib.DFT3D_INVERSE_SOLVE)
    back = inv(X)
    _finish(inv)
    inv.destroy()
    assert oracle.rel_l2(back.cpu().numpy(), x.cpu().numpy()) < TOL                     # two transforms in a row
    want = oracle.solve3d(X.cpu().numpy().astype(np.complex128), nodes)
    assert oracle.rel_l2(back.cpu().numpy(), want) < SANITY
    # the conjugate-kernel product (no flag) is NOT the inverse for these nodes
    plain = lib.Plan(*shape, sign=lib.DFT3D_INVERSE, nodes=nodes, flags=sf)
    y = plain(X)
    _finish(plain)
    plain.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), x.cpu().numpy()) > 1e-2
    # hopeless node sets and misuse are refused
    bad = [np.sort(rng.uniform(0, 1, n)) for n in shape]
    with pytest.raises(lib.Dft3dError) as e:
        lib.Plan(*shape, sign=lib.DFT3D_INVERSE, nodes=bad, flags=lib.DFT3D_INVERSE_SOLVE)
    assert e.value.status == 2
    with pytest.raises(lib.Dft3dError) as e:
        lib.Plan(*shape, sign=lib.DFT3D_FORWARD, nodes=nodes, flags=lib.DFT3D_INVERSE_SOLVE)
    assert e.value.status == 1


# ------------------------------------------------------------------ DFT3D_AUTO: the formulation chosen per axis

@pytest.mark.parametrize("split", SPLITS)
def test_auto_mode_mixes_the_formulations(lib, oracle, split):
    """Axis 0 has a length only the KDFT kernels take (100), axes 1 and 2 lengths the FFT kernels take: one plan,
    three passes through two cubes, against the oracle.  Then nonuniform nodes on axis 1 of a cube whose other axes
    are FFT lengths, with the input cube as workspace."""
    sf = _split_flag(lib, split)
    shape = (100, 256, 512)
    x = _inputs().cube(shape, "normal", 105, device="cuda")
    plan = lib.Plan(*shape, mode=lib.DFT3D_AUTO, flags=sf)
    assert plan.workspace_bytes == x.numel() * 8
    assert plan.launches == (4 if split == "fp16" else 3)      # fp16 KDFT first: one reduction over the input
    y = plan(x)
    _finish(plan)
    plan.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
    shape = (256, 128, 256)
    nodes = [None, _inputs().sorted_nodes(shape, 106)[1], None]
    x = _inputs().cube(shape, "uniform", 107, device="cuda")
    want = oracle.dft3d(x.cpu().numpy(), nodes=nodes)
    plan = lib.Plan(*shape, mode=lib.DFT3D_AUTO, nodes=nodes, flags=sf | lib.DFT3D_DESTROY_INPUT)
    assert plan.workspace_bytes == 0
    y = plan(x.clone())
    _finish(plan)
    plan.destroy()
    assert oracle.rel_l2(y.cpu().numpy(), want) < SANITY


def test_auto_mode_with_one_formulation_uses_its_schedule(lib, oracle):
    """When every axis resolves to the same formulation the plan is that formulation's plan."""
    x = _inputs().cube((256, 256, 256), "normal", 108, device="cuda")
    auto, fft = lib.Plan(256, 256, 256, mode=lib.DFT3D_AUTO), lib.Plan(256, 256, 256, mode=lib.DFT3D_FFT)
    a, b = auto(x), fft(x)
    _finish(auto)
    fft.status()
    assert torch.equal(a, b) and auto.launches == 3
    auto.destroy()
    fft.destroy()
    x = _inputs().cube((64, 96, 130), "normal", 109, device="cuda")
    auto, kd = lib.Plan(64, 96, 130, mode=lib.DFT3D_AUTO), lib.Plan(64, 96, 130, mode=lib.DFT3D_KDFT)
    a, b = auto(x), kd(x)
    _finish(auto)
    kd.status()
    assert torch.equal(a, b)
    auto.destroy()
    kd.destroy()


# ------------------------------------------------------------------ closed forms straight on the CUDA path

@pytest.mark.parametrize("mode_name", ["kdft", "fft"])
def test_closed_forms_delta_and_constant(lib, mode_name):
    """Degenerate inputs with textbook spectra, checked without the oracle: a delta at (3, 5, 7) gives the pure
    phase exp(-2 pi i (3 k0/n0 + 5 k1/n1 + 7 k2/n2)) (Eq. 14 per axis); a constant gives P at the origin and zero
    elsewhere; the inverse of the delta's spectrum is the delta."""
    shape = (256, 256, 256)
    mode = lib.DFT3D_KDFT if mode_name == "kdft" else lib.DFT3D_FFT
    plan = lib.Plan(*shape, mode=mode)
    x = torch.zeros(shape, dtype=torch.complex64, device="cuda")
    x[3, 5, 7] = 1.0
    y = plan(x)
    _finish(plan)
    k = [np.arange(n) for n in shape]
    ph = [np.exp(-2j * np.pi * s_ * k_ / n) for s_, k_, n in zip((3, 5, 7), k, shape)]
    want = ph[0][:, None, None] * ph[1][None, :, None] * ph[2][None, None, :]
    assert np.abs(y.cpu().numpy() - want).max() < 2e-6           # |X| = 1 everywhere
    inv = lib.Plan(*shape, mode=mode, sign=lib.DFT3D_INVERSE)
    back = inv(y)
    _finish(inv)
    inv.destroy()
    # (the peak is a fully coherent sum, the worst case for the tensor core's truncating accumulation: ~1e-6 per axis)
    assert (back - x).abs().max().item() < 6e-6
    c = torch.full(shape, 0.5 - 0.25j, dtype=torch.complex64, device="cuda")
    z = plan(c)
    _finish(plan)
    plan.destroy()
    P = float(np.prod(shape))
    assert abs(z[0, 0, 0].item() - P * (0.5 - 0.25j)) < 1e-5 * P
    z[0, 0, 0] = 0
    assert z.abs().max().item() < 1e-5 * P                       # leakage relative to the one peak
