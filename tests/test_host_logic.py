"""Host-side logic that needs no GPU: the C ABI loads and exports what include/glide.h declares, argument
checking, workspace sizing, error strings, and the N>1 timing aggregation of the benchmark (gloo, 2 ranks)."""
import ctypes
import os
import re
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def glide():
    from paper_2607_24788_b200 import build, glide as g
    build.build()
    g.load_library()
    return g


def declared_functions():
    text = open(os.path.join(ROOT, "include", "glide.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(glide_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(glide):
    lib = ctypes.CDLL(glide.LIB_PATH)
    names = declared_functions()
    assert {"glide_create", "glide_prefill", "glide_decode_step", "glide_destroy", "glide_workspace_bytes"} <= set(names)
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/glide.h but not exported"


def test_no_torch_types_in_the_abi():
    text = open(os.path.join(ROOT, "include", "glide.h")).read()
    assert "torch" not in text and "at::" not in text and "#include <cuda" not in text


def test_strerror(glide):
    assert glide.strerror(0) == "ok"
    assert "workspace" in glide.strerror(glide.GLIDE_ERR_WORKSPACE_TOO_SMALL)
    assert glide.strerror(12345) == "unknown status"


def _cfg(glide, **kw):
    base = dict(windows=[64, 16], batch=2, n_q_heads=8, n_kv_heads=2, head_dim=128, max_tokens=100,
                dtype=torch.bfloat16)
    base.update(kw)
    return glide.make_config(**base)


def test_workspace_bytes_scales_with_rings_and_state(glide):
    cfg, keep = _cfg(glide)
    small = glide.glide_workspace_bytes(cfg)
    cfg2, keep2 = _cfg(glide, windows=[64 + 4096, 16])
    big = glide.glide_workspace_bytes(cfg2)
    # the first layer's capacity is min(w, max_tokens) = 100: its two rings grow by (100 - 64) slots per unit;
    # the layer no longer evicts, so its state work items (and their scratch records) go away
    ring_growth = 2 * 2 * 2 * (100 - 64) * 128 * 2
    assert abs((big - small) - ring_growth) < (1 << 20) and big > small
    cfg3, keep3 = _cfg(glide, dtype=torch.float32, head_dim=64)
    assert glide.glide_workspace_bytes(cfg3) > 0


@pytest.mark.parametrize("kw,code", [
    (dict(head_dim=96), 2), (dict(n_q_heads=6, n_kv_heads=4), 2), (dict(n_q_heads=24, n_kv_heads=2), 2),
    (dict(windows=[-1, 4]), 1), (dict(max_tokens=0), 1), (dict(prefill_chunk=100), 1), (dict(decode_impl=9), 1),
    (dict(q_to_kv=[0, 0, 0, 0, 0, 1, 1, 1]), 2), (dict(q_to_kv=[0, 0, 0, 0, 1, 1, 1, 7]), 1),
    (dict(dtype=torch.float32, decode_impl=3), 2),
    (dict(merge=3), 1), (dict(merge=1, decode_impl=1), 2), (dict(merge=2, prefill_impl=1), 2), (dict(prefill_impl=7), 1),
    (dict(dtype=torch.float32, prefill_impl=2), 2),
    # ring rows of one layer must fit 32-bit indices: 4096 sequences x 2 KV heads x 2^20 slots
    (dict(batch=4096, windows=[1 << 20, 16], max_tokens=1 << 20), 2),
])
def test_invalid_configurations_are_rejected(glide, kw, code):
    cfg, keep = _cfg(glide, **kw)
    out = ctypes.c_size_t(0)
    assert glide.load_library().glide_workspace_bytes(ctypes.byref(cfg), ctypes.byref(out)) == code


def test_create_validates_before_touching_cuda(glide):
    lib = glide.load_library()
    cfg, keep = _cfg(glide)
    handle = ctypes.c_void_p()
    assert lib.glide_create(ctypes.byref(cfg), None, 1 << 30, None, ctypes.byref(handle)) == glide.GLIDE_ERR_INVALID_ARG
    assert lib.glide_create(ctypes.byref(cfg), 256, 16, None, ctypes.byref(handle)) == glide.GLIDE_ERR_WORKSPACE_TOO_SMALL
    assert lib.glide_create(ctypes.byref(cfg), 257, 1 << 40, None, ctypes.byref(handle)) == glide.GLIDE_ERR_INVALID_ARG
    assert not handle.value
    assert lib.glide_destroy(None) == glide.GLIDE_ERR_INVALID_ARG
    assert lib.glide_decode_step(None, None, None, None, None, None) == glide.GLIDE_ERR_INVALID_ARG


def test_binding_fails_loudly_without_the_library(glide, monkeypatch):
    monkeypatch.setattr(glide, "_lib", None)
    monkeypatch.setattr(glide, "LIB_PATH", "/nonexistent/libglide.so")
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        glide.load_library()


_RANK_SCRIPT = r"""
import os, sys, json
sys.path.insert(0, {root!r})
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank = dist.get_rank()
vals = bench.max_over_ranks([10.0 + rank, 5.0 - rank, 7.0], dist, torch.device("cpu"))
if rank == 0:
    print(json.dumps(dict(vals=vals, value=bench.whole_job_tokens_per_s(dist.get_world_size(), 4, 10, vals[0]))))
dist.barrier()
dist.destroy_process_group()
"""


def test_multi_rank_timing_is_max_over_ranks_and_value_sums_replicas(tmp_path):
    script = tmp_path / "rank.py"
    script.write_text(_RANK_SCRIPT.format(root=ROOT))
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2", "--master-addr", "127.0.0.1",
           "--master-port", "29731", str(script)]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    line = [l for l in r.stdout.splitlines() if l.startswith("{")][-1]
    got = json.loads(line)
    assert got["vals"] == [11.0, 5.0, 7.0]
    assert got["value"] == pytest.approx(2 * 4 * 10 / 11e-3)


def test_reference_arm_prints_one_json_line_on_cpu():
    # the reference arm (CPU oracle) on the tiny configuration; also exercises bench.py's argument handling
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "c0_tiny_f32",
                        "--steps", "4", "--warmup", "1"], capture_output=True, text=True, timeout=240)
    assert r.returncode == 0, r.stderr[-2000:]
    import json
    d = json.loads(r.stdout.strip().splitlines()[-1])
    assert d["impl"] == "reference" and d["unit"] == "tokens/s" and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0


@pytest.mark.parametrize("windows,batch,max_tokens,n_sms", [
    ([4096] * 4 + [1024] * 8 + [256] * 12 + [64] * 8, 1, 32768 + 64, 148),     # config 1: units heavier than a CTA's share
    ([4096] * 4 + [1024] * 8 + [256] * 12 + [64] * 8, 16, 16384 + 64, 148),    # config 2: hundreds of whole units per CTA
    ([1024, 512, 0, 48, 100000], 3, 5000, 148),                                # linear-only, ragged and never-evicting layers
    ([64], 1, 256, 148), ([200, 17], 2, 300, 20),
])
def test_stream_schedule_covers_every_tile_exactly_once(glide, windows, batch, max_tokens, n_sms):
    """The static schedule of the streaming decode kernel (host logic, no GPU): every 16-row tile of every unit's state
    and window is in exactly one segment, shared-memory groups and global records are numbered consistently."""
    import numpy as np
    hkv, d = 8, 128
    cfg, keep = glide.make_config(windows, batch, 32, hkv, d, max_tokens, dtype=torch.bfloat16)
    rows = glide.glide_stream_schedule(cfg, n_sms=n_sms)
    assert rows.shape[1] == 12 and len(rows) > 0
    n_units = len(windows) * batch * hkv
    seen_state = [np.zeros(d // 16, dtype=np.int32) for _ in range(n_units)]
    seen_win = {}
    for cta, warp, unit, layer, nst, st0, nw, w0, gsz, slot, part, nparts in rows.tolist():
        assert 0 <= cta < n_sms and 0 <= warp < 8 and 0 <= unit < n_units and layer == unit // (batch * hkv)
        cap = min(windows[layer], max_tokens)
        tiles = (cap + 15) // 16
        evicts = windows[layer] < max_tokens
        assert nst >= 0 and nw >= 0 and st0 + nst <= (d // 16 if evicts else 0) and w0 + nw <= tiles
        seen_state[unit][st0:st0 + nst] += 1
        seen_win.setdefault(unit, np.zeros(tiles, dtype=np.int32))[w0:w0 + nw] += 1
    for unit in range(n_units):
        layer = unit // (batch * hkv)
        evicts = windows[layer] < max_tokens
        assert unit in seen_win, f"unit {unit} has no segment"
        assert (seen_win[unit] == 1).all(), f"window tiles of unit {unit}"
        assert (seen_state[unit] == (1 if evicts else 0)).all(), f"state tiles of unit {unit}"
    # groups: the segments of one unit inside one CTA carry its size and distinct slots; records: 0 .. n_parts - 1
    by_cta_unit, by_unit = {}, {}
    for r in rows.tolist():
        by_cta_unit.setdefault((r[0], r[2]), []).append(r)
        by_unit.setdefault(r[2], []).append(r)
    for (cta, unit), rs in by_cta_unit.items():
        sizes = {r[8] for r in rs}
        if sizes != {1}:
            assert sizes == {len(rs)} and len({r[9] for r in rs}) == len(rs) and min(r[9] for r in rs) >= 0
        assert len({r[1] for r in rs}) == len(rs) or sizes == {1}, "one segment per warp in a group"
    for cta in {r[0] for r in rows.tolist()}:
        slots = [r[9] for r in rows.tolist() if r[0] == cta and r[9] >= 0]
        assert len(slots) == len(set(slots)), "record slots of a CTA are distinct"
    for unit, rs in by_unit.items():
        nparts = {r[11] for r in rs}
        assert len(nparts) == 1
        n = nparts.pop()
        parts = sorted({r[10] for r in rs})
        assert parts == ([-1] if n == 1 else list(range(n)))


def test_stream_schedule_refuses_what_the_kernel_does_not_run(glide):
    cfg, keep = glide.make_config([64], 1, 4, 4, 64, 128, dtype=torch.bfloat16)
    with pytest.raises(glide.GlideError) as e:
        glide.glide_stream_schedule(cfg)
    assert e.value.code == glide.GLIDE_ERR_UNSUPPORTED


def test_stream_schedule_balances_the_warps_of_a_cta(glide):
    """Config 1: inside every CTA the heaviest warp (in the schedule's own weights: 15 per state tile, 10 per window
    tile, 27 per segment) is at most one window tile and one segment above the CTA's mean warp, and no unit is cut into
    more records than the whole-stack problem needs (a unit of a 4096-token window is about 2.2 CTA shares)."""
    import numpy as np
    windows = [4096] * 4 + [1024] * 8 + [256] * 12 + [64] * 8
    cfg, keep = glide.make_config(windows, 1, 32, 8, 128, 32768 + 64, dtype=torch.bfloat16)
    rows = glide.glide_stream_schedule(cfg)
    w = rows[:, 4] * 15 + rows[:, 6] * 10 + 27
    warp = rows[:, 0] * 8 + rows[:, 1]
    per_warp = np.bincount(warp, weights=w, minlength=148 * 8).reshape(148, 8)
    assert (per_warp.max(axis=1) <= per_warp.sum(axis=1) / 8 + 10 + 27 + 15).all()
    assert rows[:, 11].max() <= 5
    assert per_warp.sum(axis=1).max() <= 1.1 * per_warp.sum(axis=1).mean()


def test_stream_schedule_limits_the_records_of_a_small_problem(glide):
    """One long-window layer at batch 1 leaves a CTA only a few dozen tiles: its units are then cut into at most about
    eight records each (the merge reads them a few at a time); a problem with hundreds of tiles per CTA keeps all SMs."""
    cfg, keep = glide.make_config([4096], 1, 32, 8, 128, 8192, dtype=torch.bfloat16)
    rows = glide.glide_stream_schedule(cfg)
    assert rows[:, 11].max() <= 10 and len(set(rows[:, 0].tolist())) <= 8 * 8 + 8
    cfg, keep = glide.make_config([131072], 1, 32, 8, 128, 131072 + 64, dtype=torch.bfloat16)
    rows = glide.glide_stream_schedule(cfg)
    assert len(set(rows[:, 0].tolist())) == 148
