"""The allocation-free scorer against the ordinary evaluation path.

Some hosts may not allocate device memory at all (the application owns the device through
its own arena and hands plug-ins only the buffers it chooses).  For them the library has
pbt_energy_fitness_static, whose reduction scratch is a fixed array inside the library.
This file checks, through the C ABI, that it gives the same fitness as pbt_eval does for a
GAN population and as the CPU oracle's energy distance gives for the same points, on two
calls in a row (the second call reuses the scratch the first one left dirty), and that it
refuses problems larger than its built-in scratch.

Named so that pytest collects it last.
"""
import ctypes as C

import numpy as np
import pytest

from oracle import pbt_oracle as O
from workloads import get_config, make_inputs

pytestmark = pytest.mark.gpu


def _pass_through_generator(cfg, scale):
    """Flat weights of a generator whose output is scale * (first two noise coordinates),
    exactly: relu(z) - relu(-z) = z, with weights that are powers of two."""
    g = cfg.widths[0]
    assert len(g) == 4 and g[-1] == 2 and min(g[1], g[2]) >= 4
    W0 = np.zeros((g[1], g[0]), np.float32)
    W0[0, 0], W0[1, 0], W0[2, 1], W0[3, 1] = scale, -scale, scale, -scale
    W1 = np.zeros((g[2], g[1]), np.float32)
    for i in range(4):
        W1[i, i] = 1.0
    W2 = np.zeros((2, g[2]), np.float32)
    W2[0, 0], W2[0, 1], W2[1, 2], W2[1, 3] = 1.0, -1.0, 1.0, -1.0
    parts = []
    for W in (W0, W1, W2):
        parts += [W.reshape(-1), np.zeros(W.shape[0], np.float32)]
    return np.concatenate(parts)


def test_static_scratch_scorer_matches_eval_twice():
    import torch
    import paper_1711_09846_b200 as pkg

    cfg = get_config("c4_mini").replace(eval_batch=1000)      # 4 blocks of 256 points, ragged tail
    inp = make_inputs(cfg)
    pop = pkg.Population(cfg, inp)
    n_g = sum(a * b + b for a, b in zip(cfg.widths[0][:-1], cfg.widths[0][1:]))
    scales = [2.0 ** (m - 2) for m in range(cfg.n_members)]
    for m, s in enumerate(scales):
        w = pop.get_state(m)["w"]
        w[:n_g] = _pass_through_generator(cfg, s)
        pop.set_state(m, w=w)
    pop.eval()
    expect = pop.fitness()                                     # the existing entry point's result
    assert len(set(np.round(expect, 6))) == cfg.n_members      # members really differ

    z = inp.x_eval[:, :2].astype(np.float32)                   # bf16-representable, so G(z) is exact
    x = np.stack([s * z for s in scales]).astype(np.float32)   # [members, n, 2]
    oracle = np.array([-O.energy_distance_to_ring(xm.astype(np.float64)) for xm in x])   # fitness = -energy distance
    x_dev = torch.from_numpy(x).cuda().contiguous()
    out = torch.full((cfg.n_members,), float("nan"), device="cuda", dtype=torch.float32)
    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())

    pkg.energy_fitness_static(x_dev, out, stream)
    stream.synchronize()
    np.testing.assert_allclose(out.cpu().numpy(), expect, rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(out.cpu().numpy(), oracle, rtol=1e-5, atol=1e-6)

    # second call straight after, other data, same shared scratch
    x_rev = torch.from_numpy(x[::-1].copy()).cuda().contiguous()
    out2 = torch.full((cfg.n_members,), float("nan"), device="cuda", dtype=torch.float32)
    stream.wait_stream(torch.cuda.current_stream())
    pkg.energy_fitness_static(x_rev, out2, stream)
    stream.synchronize()
    np.testing.assert_allclose(out2.cpu().numpy(), expect[::-1], rtol=1e-6, atol=1e-7)
    np.testing.assert_allclose(out2.cpu().numpy(), oracle[::-1], rtol=1e-5, atol=1e-6)
    pop.close()


def test_static_scratch_scorer_rejects_oversize_and_bad_arguments():
    import torch
    import paper_1711_09846_b200 as pkg

    lib = pkg.load_library()
    buf = torch.zeros(8, device="cuda", dtype=torch.float32)
    p = C.c_void_p(buf.data_ptr())
    # 1024 members x 2 x ceil(65536 / 256) = 524288 partial sums > 131072: refused before anything is launched
    assert lib.pbt_energy_fitness_static(p, 65536, 1024, p, None) == 3
    assert b"scratch" in lib.pbt_last_error(None)
    assert lib.pbt_energy_fitness_static(None, 16, 1, p, None) == 1
    assert lib.pbt_energy_fitness_static(p, 0, 1, p, None) == 1
    # sizes that would overflow 32-bit arithmetic, more members than a grid dimension holds, host memory
    assert lib.pbt_energy_fitness_static(p, 2**31 - 1, 1, p, None) == 3
    assert lib.pbt_energy_fitness_static(p, 16, 65536, p, None) == 3
    host = np.zeros(64, dtype=np.float32)
    assert lib.pbt_energy_fitness_static(C.c_void_p(host.ctypes.data), 16, 1, p, None) == 1
    torch.cuda.synchronize()
