"""GPU parity on seeded random configurations: dtype, head_dim, group size, batch, number of layers, windows (0, tiny,
around the tile sizes, longer than the sequence), several prefill calls, decode steps, merge, kernel choices.
Complements the hand-picked cases of test_gpu_parity.py; every case is reproducible from its seed."""
import random

import pytest
import torch

from tests.parity_util import run_case

pytestmark = pytest.mark.gpu

BF16, F32 = torch.bfloat16, torch.float32
WINDOWS = [0, 1, 2, 7, 15, 16, 17, 31, 48, 64, 100, 129, 300, 777, 1 << 20]


def draw(seed):
    rng = random.Random(seed)
    dtype = rng.choice([BF16, BF16, BF16, F32])
    d = rng.choice([128, 128, 64]) if dtype == BF16 else 64
    G, Hkv, B = rng.choice([1, 2, 4, 8]), rng.choice([1, 2, 3]), rng.choice([1, 2, 3, 5])
    windows = [rng.choice(WINDOWS) for _ in range(rng.choice([1, 2, 3, 6, 12]))]
    calls = [rng.choice([1, 5, 16, 33, 64, 100, 257]) for _ in range(rng.choice([0, 1, 2, 3]))]
    n_dec = rng.choice([1, 3, 9, 20])
    merge = rng.choice([0, 0, 0, 1, 2])
    kw = dict(merge=merge, prefill_chunk=rng.choice([16, 32, 96, 256]))
    if dtype == BF16 and d == 128 and merge == 0:
        kw["decode_impl"] = rng.choice([0, 0, 1, 2, 3])
        kw["prefill_impl"] = rng.choice([0, 0, 1, 2, 3])
    amp = 1.0 if dtype == F32 else d ** -0.5 * rng.choice([1, 4, 10])
    return dict(windows=windows, B=B, H=G * Hkv, Hkv=Hkv, d=d, dtype=dtype, calls=calls, n_dec=n_dec, amp=amp, kw=kw)


@pytest.mark.parametrize("seed", range(100, 116))
def test_random_configuration(seed):
    c = draw(seed)
    run_case(c["windows"], c["B"], c["H"], c["Hkv"], c["d"], c["dtype"], c["calls"], c["n_dec"], amp=c["amp"], seed=seed,
             **c["kw"])
