"""Every output element of the full-size problems, not a sample of rows.

The oracle can afford only a few dozen rows of an 8192^3 problem, so the full-size parity tests compare
sampled rows.  What those leave uncovered -- a tile of the 13.8-wave schedule that is dropped or written
to the wrong place, a tile group walked backwards, a K cut of the last wave that loses a k-block -- is
caught here by a Freivalds-style product check with the identity activation, which costs O(MN) on the
host: for every 256-column block j a random sign vector r_j supported on that block,

    (Y r_j)[m]  against  X (W^T r_j) + b . r_j        (float64 on the host),

one checked value per (row, column block).  The bound is not statistical: each stored output is off by at
most its rounding (2^-9 relative for bf16 storage) plus the fp32 accumulation, so the product may differ
by at most that times the sum of |y| over the block.
"""
import dataclasses

import numpy as np
import pytest

from paper_2511_01884_b200 import binding as B
from paper_2511_01884_b200 import workloads as wk

import parity_util as pu

pytestmark = pytest.mark.gpu

BLOCK = 256


def _block_products(g, inp, N, rng):
    """(Y r_j)[m] from the GPU result and its float64 reference, both [M, N / BLOCK], and sum |y| per block."""
    nb = N // BLOCK
    r = rng.choice([-1.0, 1.0], size=N)
    X = inp["X"].astype(np.float64)
    W = inp["W"].astype(np.float64)
    V = (W * r[:, None]).reshape(nb, BLOCK, -1).sum(1)              # [nb, K]: W^T r_j for every block
    want = X @ V.T
    if inp["b"] is not None:
        want += (inp["b"].astype(np.float64) * r).reshape(nb, BLOCK).sum(1)[None, :]
    got = (g * r[None, :]).reshape(g.shape[0], nb, BLOCK).sum(2)
    mass = np.abs(g).reshape(g.shape[0], nb, BLOCK).sum(2)
    return got, want, mass


@pytest.mark.parametrize("name,kernel,rel", [("c3", B.FORGE_KERNEL_BF16_TCGEN05, 2.0 ** -9 + 1e-5),
                                             ("c2", B.FORGE_KERNEL_F32_FFMA, 1e-5),
                                             ("c2t", B.FORGE_KERNEL_F32_TF32X3, 1e-5)])
def test_every_tile_of_the_full_size_schedule(name, kernel, rel):
    base = {**wk.WORKLOADS, **wk.EXTRA_WORKLOADS}[name]
    wl = dataclasses.replace(base, name=name + "_identity", act=wk.ACT_IDENTITY, scale=1.0)
    inp = wk.make_inputs(wl)
    g, plan = pu.run_gpu(wl, inp)
    assert plan["kernel"] == kernel
    assert np.isfinite(g).all()
    got, want, mass = _block_products(g, inp, wl.N, np.random.default_rng(7))
    excess = np.abs(got - want) - rel * mass
    worst = np.unravel_index(np.argmax(excess), excess.shape)
    assert excess.max() <= 0.0, (f"row {worst[0]}, columns {BLOCK * worst[1]}..: product off by "
                                 f"{abs(got[worst] - want[worst]):.3e}, allowed {rel * mass[worst]:.3e}")
    # the check can see a single wrong element: move one reference value by the size of one output and it must trip
    want2 = want.copy()
    want2[4097 % wl.M, 7 % want.shape[1]] += float(np.sqrt(np.mean(g * g)))
    assert (np.abs(got - want2) - rel * mass).max() > 0.0
