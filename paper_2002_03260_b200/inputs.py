"""Seeded synthetic inputs shaped like the paper's workloads (cubes of complex samples).

Shared by the tests, the smoke check and the bench.  Holds no arithmetic of the transform itself:
only random draws, and for the "exponentials" workload the sample-domain signal whose spectrum is
known in closed form.  The paper's experiments use cubes of unstated contents (Table I sizes), so
seeded random data of those shapes stands in for them.
"""
import numpy as np
import torch


def cube(shape, dist, seed, device="cpu"):
    """complex64 tensor [n0, n1, n2]; real and imaginary parts iid `dist` in {"uniform", "normal"}.

    uniform = U(-1, 1), normal = N(0, 1).  On a CUDA device the draw uses torch's CUDA generator
    (plane by plane, so no large temporaries); on the CPU it uses numpy's PCG64.  The two streams
    differ; a test always hands the bytes it generated to both the oracle and the GPU path.
    """
    shape = tuple(int(s) for s in shape)
    dev = torch.device(device)
    if dev.type == "cpu":
        r = np.random.default_rng(seed)
        buf = np.empty(shape + (2,), dtype=np.float32)
        flat = buf.reshape(shape[0], -1)
        for a in range(shape[0]):
            if dist == "uniform":
                flat[a] = r.random(flat.shape[1], dtype=np.float32) * 2.0 - 1.0
            elif dist == "normal":
                flat[a] = r.standard_normal(flat.shape[1], dtype=np.float32)
            else:
                raise ValueError(dist)
        return torch.view_as_complex(torch.from_numpy(buf))
    g = torch.Generator(device=dev)
    g.manual_seed(seed)
    x = torch.empty(shape, dtype=torch.complex64, device=dev)
    xr = torch.view_as_real(x)
    for a in range(shape[0]):
        if dist == "uniform":
            xr[a].uniform_(-1.0, 1.0, generator=g)
        elif dist == "normal":
            xr[a].normal_(0.0, 1.0, generator=g)
        else:
            raise ValueError(dist)
    return x


def sorted_nodes(shape, seed):
    """Three independent ascending arrays of nodes in [0, 1) (float64), one per axis."""
    r = np.random.default_rng(seed)
    return tuple(np.sort(r.random(int(n))) for n in shape)


def exponentials(shape, count, seed, noise_std, noise_seed, device="cpu"):
    """Sum of `count` unit-amplitude complex exponentials with distinct integer frequency triples and
    seeded phases, plus N(0, noise_std^2) noise on each real and imaginary component.

    Returns (x, freqs[count, 3], phases[count]).  Built plane by plane from three 1D float64 phasor
    vectors per exponential (separable), cast to float32 once.
    """
    shape = tuple(int(s) for s in shape)
    r = np.random.default_rng(seed)
    freqs = set()
    while len(freqs) < count:
        freqs.add(tuple(int(r.integers(0, n)) for n in shape))
    freqs = np.array(sorted(freqs), dtype=np.int64)
    phases = r.random(count) * 2.0 * np.pi
    dev = torch.device(device)
    x = cube(shape, "normal", noise_seed, device=dev)
    torch.view_as_real(x).mul_(noise_std)
    ax = [torch.arange(n, dtype=torch.float64, device=dev) for n in shape]
    for a in range(shape[0]):
        plane = torch.zeros(shape[1:], dtype=torch.complex128, device=dev)
        for e in range(count):
            f = freqs[e]
            c0 = np.exp(1j * (2.0 * np.pi * ((f[0] * a) % shape[0]) / shape[0] + phases[e]))
            v1 = torch.exp(2j * np.pi * ((f[1] * ax[1]) % shape[1]) / shape[1])
            v2 = torch.exp(2j * np.pi * ((f[2] * ax[2]) % shape[2]) / shape[2])
            plane += complex(c0) * torch.outer(v1, v2)
        x[a] += plane.to(torch.complex64)
    return x, freqs, phases


def stratified_indices(n, count, seed, forced=()):
    """`count` indices, the i-th drawn from [i*n/count, (i+1)*n/count), plus 0, n-1 and `forced`; sorted, unique."""
    r = np.random.default_rng(seed)
    count = min(count, n)
    edges = np.linspace(0, n, count + 1).astype(np.int64)
    idx = [int(r.integers(edges[i], max(edges[i] + 1, edges[i + 1]))) for i in range(count)]
    idx += [0, n - 1] + [int(f) for f in forced]
    return np.unique(np.array(idx, dtype=np.int64))
