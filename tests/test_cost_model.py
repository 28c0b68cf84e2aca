"""Byte accounting and cost model against the numbers the paper prints."""
import os

import pytest

from paper_2607_24788_b200 import configs as C

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
MiB = 1 << 20


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [l.split() for l in f if l.strip() and not l.startswith("#")]


@pytest.mark.parametrize("row", _rows("kv_io_table1.txt"))
def test_table1_kv_io_column(row):
    _, d1, d2, d3, mib = row
    windows = C.blockwise_windows(1024, (int(d1), int(d2), int(d3)), (10, 12, 10))
    assert len(windows) == 32
    got = C.kv_io_bytes_per_token(windows) / MiB
    assert round(got) == int(mib)          # the table prints whole MiB
    if int(d2) != 960:
        assert got == int(mib)             # exact for every row but 15w/16 (42.75 MiB, printed 43)


@pytest.mark.parametrize("row", _rows("kv_io_fig4.txt"))
def test_fig4_kv_io(row):
    _, tokens, frac, mib = row
    windows = [int(int(tokens) * float(frac))] * 32
    assert C.kv_io_bytes_per_token(windows) / MiB == float(mib)


def test_speedup_identity_and_limit():
    # Sec. III-C: cost(0,0,0) / cost(0, alpha w, w) == 1 + (1+alpha)/((2+3d/w) - alpha), at most 3
    for L, w, d, a in [(32, 1024, 128, 0.5), (30, 64, 128, 0.0), (33, 4096, 64, 1.0), (12, 20000, 128, 15 / 16)]:
        ratio = (L * w * d + L * d * d) / C.blockwise_cost(L, w, d, a)
        assert ratio == pytest.approx(C.theoretical_speedup(a, w, d), rel=1e-12)
    assert C.theoretical_speedup(1.0, 1e12, 128) == pytest.approx(3.0, rel=1e-6)
    assert C.theoretical_speedup(1.0, 1024, 128) < 3.0


def test_config_windows():
    assert sum(C.C1.windows) == 28160 and len(C.C1.windows) == 32
    assert sum(C.C2_UNIFORM.windows) == 32768
    assert sum(C.C3.windows) == 277504
    w4 = list(C.C4.windows)
    assert sum(w4) == 25680 and w4[0] == 4096 and w4[-1] == 32 and all(x % 16 == 0 for x in w4)
    assert w4[:6] == [4096, 3440, 2896, 2432, 2048, 1728]
    assert list(C.P1.windows) == [1024] * 10 + [512] * 12 + [0] * 10


def test_decode_step_bytes():
    # window term and state term of the roofline formula, config 1 at 32K context
    assert C.decode_step_bytes(C.C1, 32768) == 149_946_368
    s = C.GlideShape("x", 1, 1, 4, 4, 64, (8,), 0, 0, "f32")
    # n = 3 < w: reads 4 slots (incl. the current row), no state traffic
    assert C.decode_step_bytes(s, 3) == 2 * 4 * 4 * 64 * 4 + 2 * 4 * 64 * 4 + (8 + 8) * 64 * 4
    # n = 8 >= w: 8 slots + state read/write
    assert C.decode_step_bytes(s, 8) == 2 * 8 * 4 * 64 * 4 + 2 * (4 * 64 * 64 + 4 * 64) * 4 + 2 * 4 * 64 * 4 + 16 * 64 * 4


def test_blockwise_allocation_search():
    # Algorithm 1: early block delta 0, last block delta w, the middle block's delta picked by the caller's score
    assert C.three_block_split(32) == [11, 11, 10] and C.three_block_split(30) == [10, 10, 10]
    assert C.blockwise_delta_candidates(1024) == [0, 512, 960, 1024]
    seen = []

    def acc(windows):
        seen.append(list(windows))
        return {1024: 0.70, 512: 0.69, 64: 0.71, 0: 0.40}[windows[15]]

    windows, delta, scores = C.blockwise_allocate(32, 1024, acc, split=(10, 12, 10))
    assert delta == 960 and windows == [1024] * 10 + [64] * 12 + [0] * 10
    assert scores == {0: 0.70, 512: 0.69, 960: 0.71, 1024: 0.40}
    assert len(seen) == 4 and all(s[:10] == [1024] * 10 and s[22:] == [0] * 10 for s in seen)
    # equal scores: the allocation that reads less of the cache
    _, delta, _ = C.blockwise_allocate(30, 1024, lambda ws: 1.0)
    assert delta == 1024
    # the chosen row reproduces the KV I/O the table prints for it (0, 15w/16, w): 43 MiB
    assert round(C.kv_io_bytes_per_token(windows) / MiB) == 43
    with pytest.raises(ValueError):
        C.blockwise_allocate(32, 1024, acc, split=(10, 10, 10))
