"""The synthetic input generator: addressable, deterministic, right distribution, exact in the I/O dtype."""
import torch

from paper_2607_24788_b200 import synth


def test_addressable_and_deterministic():
    w = synth.Workload(3, 4, 2, 8, 2, 64, torch.bfloat16, 0.125)
    q, k, v = w.qkv(range(4), range(2), range(50))
    assert q.shape == (4, 2, 50, 8, 64) and k.shape == (4, 2, 50, 2, 64) and q.dtype == torch.bfloat16
    q2, k2, v2 = w.qkv([2], [1], [7, 49])
    assert torch.equal(q2[0, 0, 0], q[2, 1, 7]) and torch.equal(k2[0, 0, 1], k[2, 1, 49]) and torch.equal(v2[0, 0, 0], v[2, 1, 7])
    qd, kd, vd = w.decode_qkv(49)
    assert torch.equal(qd, q[:, :, 49]) and torch.equal(vd, v[:, :, 49])
    other = synth.Workload(4, 4, 2, 8, 2, 64, torch.bfloat16, 0.125).qkv(range(1), range(1), range(4))[0]
    assert not torch.equal(other, q[:1, :1, :4])
    assert not torch.equal(k[..., :2, :], q[..., :2, :])


def test_distribution():
    w = synth.Workload(0, 1, 1, 32, 8, 128, torch.float32, 1.0)
    q = w.qkv([0], [0], range(256))[0].double()
    assert abs(float(q.mean())) < 5e-3 and abs(float(q.std()) - 1.0) < 5e-3
    assert abs(float((q ** 4).mean()) - 3.0) < 0.1
    # neighbouring features / tokens are uncorrelated
    assert abs(float((q[..., :-1] * q[..., 1:]).mean())) < 5e-3
    assert abs(float((q[0, 0, :-1] * q[0, 0, 1:]).mean())) < 5e-3


def test_table_is_exact_in_dtype():
    t = synth.normal_table(128 ** -0.5, torch.bfloat16)
    assert t.dtype == torch.bfloat16 and t.shape == (65536,)
    assert torch.equal(t.float().to(torch.bfloat16), t)
    assert float(t[0]) < -0.3 and float(t[-1]) > 0.3 and torch.all(t[1:] >= t[:-1])
