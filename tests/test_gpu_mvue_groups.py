"""The MVUE group rule of the kernel against the oracle's, group by group, on explicit uniforms.

Whole-tensor parity reaches the rule's corner cases only by luck (u = 1 - 2^-24 has probability 6e-8 per group).
Here groups and uniforms are chosen: every u that makes a sampling point land on, just below or just above a
cumulative sum; u = 0 and u = 1 - 2^-24; zero magnitudes in every position; ties for the maximum; magnitudes 2^17
apart (sums that round); the clipped / unclipped boundary m_x = rest.  Positions and fp32 values must match bit for bit.
"""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(2024)
    groups = []
    alphabet = np.array([0.0, -0.0, 1.0, -1.0, 2.0, 0.5, 3.0, 1.5, 2.0 ** -17, -(2.0 ** -17), 2.0 ** -126, 7.0, 1.0078125, 96.0],
                        dtype=np.float32)
    idx = np.stack(np.meshgrid(*[np.arange(len(alphabet))] * 4, indexing="ij"), -1).reshape(-1, 4)
    groups.append(alphabet[idx[rng.choice(len(idx), 6000, replace=False)]])            # structured: zeros, ties, tiny, huge ratios
    groups.append(rng.standard_normal((6000, 4)).astype(np.float32) * 0.01)             # gradient-like
    g = rng.standard_normal((3000, 4)).astype(np.float32)
    g[:, 3] = np.abs(g[:, :3]).sum(1) * rng.choice([1.0, -1.0], 3000)                   # near the clipped / unclipped boundary
    groups.append(g)
    a = synth.bf16_bits_to_f32(synth.to_bf16_bits(np.concatenate(groups)))
    n = len(a)
    # uniforms: the ends, random ones, and for every group the u that puts u*h (or u*h + h) next to a cumulative sum
    ks = [np.zeros(n, np.uint32), np.full(n, (1 << 24) - 1, np.uint32), np.full(n, 1 << 23, np.uint32),
          rng.integers(0, 1 << 24, n, dtype=np.uint32), rng.integers(0, 1 << 24, n, dtype=np.uint32)]
    m = np.abs(a).astype(np.float64)
    tot = m.sum(1)
    for target in (m[:, 0], m[:, 0] + m[:, 1], m[:, 0] + m[:, 1] + m[:, 2]):
        for h in (tot / 2, tot - m.max(1)):                                              # unclipped / clipped interval length
            with np.errstate(divide="ignore", invalid="ignore"):
                for t in (target, target - h):
                    u0 = np.where(h > 0, t / h, 0.0)
                    k0 = np.clip(np.nan_to_num(u0) * (1 << 24), 0, (1 << 24) - 1)
                    for d in (-1, 0, 1):
                        ks.append(np.clip(np.floor(k0) + d, 0, (1 << 24) - 1).astype(np.uint32))
    return a, ks


def test_group_rule_matches_the_oracle_on_chosen_uniforms():
    from paper_2409_09099_b200 import binding as B
    ctx = B.Context(0)
    a, ks = _cases()
    n = len(a)
    a_dev = torch.from_numpy(synth.to_bf16_bits(a).view(np.int16)).to(DEV).view(torch.bfloat16)
    pos = torch.empty(n, dtype=torch.int32, device=DEV)
    val = torch.empty((n, 2), dtype=torch.float32, device=DEV)
    opos, oval = np.empty(2, np.int32), np.empty(2, np.float32)
    checked = 0
    for k in ks:
        ctx.debug_mvue_groups(a_dev, torch.from_numpy(k.view(np.int32)).to(DEV), pos, val)
        gp, gv = pos.cpu().numpy(), val.cpu().numpy()
        u = k.astype(np.float32) * np.float32(2.0 ** -24)
        for i in range(n):
            p, v = orc.mvue_group(a[i], u[i])
            assert gp[i] == (p[0] | (p[1] << 2)), (a[i], k[i], gp[i], p)
            assert gv[i].view(np.uint32).tolist() == v.view(np.uint32).tolist(), (a[i], k[i], gv[i], v)
        checked += n
    assert checked > 500000
    assert ctx.poll_device_status() == 0
    ctx.close()
