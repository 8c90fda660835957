"""The allocation-free entry point, dft3d_kdft_execute_static, against the plan-based path.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has already run
every other test.  It is meant for callers that cannot call cudaMalloc where they need the transform (allocator
off limits, all device memory owned by someone else); here the test plays that caller: it owns the tables, the
input and the output, and the library may only use its built-in scratch array.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")

pytestmark = pytest.mark.gpu

SANITY = 5e-6   # the 3D-transform bound the other GPU tests use


def _tables(dft, shape, sign=-1, scale_inverse=False):
    out = []
    for n in shape:
        hi, lo = dft.generate_real_table(n, sign=sign, scale=(1.0 / n if scale_inverse else 1.0))
        out.append(torch.from_numpy(np.stack([hi, lo])).cuda())
    return out


def test_static_entry_point_matches_plan_twice_in_a_row():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2002_03260_b200 as dft
    from paper_2002_03260_b200 import inputs
    from oracle import oracle

    first = None
    for shape, seed in (((128, 128, 128), 71), ((64, 128, 256), 72)):    # two calls in a row share the scratch array
        x = inputs.cube(shape, "normal", seed, device="cuda")
        tables = _tables(dft, shape)
        out = torch.empty_like(x)
        before = torch.cuda.memory_allocated()
        dft.kdft_execute_static(x, out, tables)
        assert torch.cuda.memory_allocated() == before
        # torch's counter sees only torch's own allocator; the driver's free-memory figure sees a cudaMalloc from
        # anywhere in the process.  Compare it across a second call (the first one on a device may load kernels),
        # with no torch allocation in between.
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        dft.kdft_execute_static(x, out, tables)
        assert torch.cuda.mem_get_info()[0] == free_before
        # and against the float64 oracle directly, not only against the plan-based path
        assert oracle.rel_l2(out.cpu().numpy(), oracle.dft3d(x.cpu().numpy())) < SANITY
        plan = dft.Plan(*shape, mode=dft.DFT3D_KDFT, flags=dft.DFT3D_SPLIT_TF32)  # same TF32 tables and kernel as the static entry
        want = plan(x)
        torch.cuda.synchronize()
        plan.status()
        plan.destroy()
        err = oracle.rel_l2(out.cpu().numpy(), want.cpu().numpy())
        assert err < SANITY, (shape, err)
        assert torch.equal(out, want)       # same kernels, same tables, same order: identical bits
        if first is None:
            first = (x, out.clone(), tables)
    # the first problem again, after the scratch held another problem's data
    x, want, tables = first
    again = torch.empty_like(x)
    dft.kdft_execute_static(x, again, tables)
    assert torch.equal(again, want)


def test_static_entry_point_rejects_what_it_cannot_hold():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import paper_2002_03260_b200 as dft
    shape = (256, 128, 128)      # 4 Mi points: twice the static scratch
    x = torch.zeros(shape, dtype=torch.complex64, device="cuda")
    out = torch.empty_like(x)
    tables = [torch.zeros((2, 2 * n, 2 * n), device="cuda") for n in shape]
    with pytest.raises(dft.Dft3dError) as e:
        dft.kdft_execute_static(x, out, tables)
    assert e.value.status == 2 and "exceed the static scratch" in str(e.value)
    small = x[:64, :64, :100].contiguous()      # 100 is not a multiple of 64
    with pytest.raises(dft.Dft3dError) as e:
        dft.kdft_execute_static(small, torch.empty_like(small),
                                [torch.zeros((2, 2 * n, 2 * n), device="cuda") for n in small.shape])
    assert e.value.status == 2
    with pytest.raises(ValueError):             # the binding refuses an output of another shape before any kernel runs
        dft.kdft_execute_static(small, out, tables)
