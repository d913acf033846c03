"""Pins for the oracle's projection, beta and compression against what the paper fixes.

Eq. 4 (S_soft), Theorem 4.1 and its proof (closed forms, continuity, projection),
Eq. 5 (beta as the MSE minimiser).  None of these checks re-types the oracle's
own formula: they use hand-worked groups, invariants, brute force and the
textbook soft-threshold operator.
"""
import itertools
import os

import numpy as np
import pytest

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x):
    return synth.to_bf16_bits(np.asarray(x, np.float32))


def _golden_groups():
    rows = []
    with open(os.path.join(GOLDEN, "s_soft_groups.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            a, s, p = [part.split() for part in line.split("|")]
            rows.append(([float(v) for v in a], [float(v) for v in s], [int(v) for v in p]))
    return rows


def test_s_soft_hand_worked_groups():
    for a, s, _ in _golden_groups():
        got = orc.s_soft(_bits([a]))[0]
        assert np.array_equal(got, np.asarray(s, np.float32)), (a, s, got)
        assert not np.signbit(got[got == 0]).any(), "pruned entries are +0"


def test_compress_hand_worked_groups():
    for a, s, kept in _golden_groups():
        row = a * 4                                     # K = 16: one metadata word
        vals, meta, dense = orc.project_compress(_bits([row]), 1.0)
        for g in range(4):
            nib = (int(meta[0, 0]) >> (4 * g)) & 0xF
            assert (nib & 3, nib >> 2) == tuple(kept), (a, nib)
            v = synth.bf16_bits_to_f32(vals[0, 2 * g:2 * g + 2])
            assert np.array_equal(v, np.asarray([s[kept[0]], s[kept[1]]], np.float32))
        assert np.array_equal(synth.bf16_bits_to_f32(dense[0]), np.asarray(s * 4, np.float32))


def test_s_soft_threshold_brute_force():
    """t is the value with at most 2 magnitudes above it and at least 3 at or above it."""
    rng = np.random.default_rng(11)
    W = synth.gaussian_bf16(11, (1000, 100), 0.02)
    # add ties and zeros
    Wf = synth.bf16_bits_to_f32(W)
    mask = rng.random(Wf.shape) < 0.2
    Wf[mask] = np.round(Wf[mask] * 64) / 64
    W = _bits(Wf)
    Wf = synth.bf16_bits_to_f32(W).astype(np.float64)
    S = orc.s_soft(W).astype(np.float64)
    A = Wf.reshape(-1, 4)
    Sg = S.reshape(-1, 4)
    M = np.abs(A)
    t = np.sort(M, axis=1)[:, 1]
    assert ((M > t[:, None]).sum(1) <= 2).all() and ((M >= t[:, None]).sum(1) >= 3).all()
    # textbook soft-threshold (the l1 proximal operator) with per-group lambda = t
    expect = np.sign(A) * np.maximum(M - t[:, None], 0.0)
    # one fp32 subtraction of bf16 magnitudes vs the exact difference
    assert np.allclose(Sg, expect, rtol=2.0 ** -23, atol=0)
    assert ((Sg != 0).sum(1) <= 2).all()


def test_s_soft_all_patterns_small_alphabet():
    alphabet = [0.0, 1.0, -1.0, 2.0, -3.0]
    groups = np.array(list(itertools.product(alphabet, repeat=4)), np.float32)
    S = orc.s_soft(_bits(groups))
    for a, s in zip(groups.astype(np.float64), S.astype(np.float64)):
        m = sorted(abs(a))
        t = m[1]
        for ai, si in zip(a, s):
            assert si == (np.sign(ai) * max(abs(ai) - t, 0.0))
        assert (s != 0).sum() <= 2


def test_s_soft_is_projection_and_equivariant():
    W = synth.gaussian_bf16(5, (64, 64), 1.0)
    Wf = synth.bf16_bits_to_f32(W)
    # keep magnitudes on a coarse grid so that differences stay exactly representable in bf16
    Wf = np.round(Wf * 8) / 8
    W = _bits(Wf)
    S = orc.s_soft(W)
    assert np.array_equal(synth.bf16_bits_to_f32(_bits(S)), S), "test premise: S is bf16-representable"
    # Theorem 4.1: a projection is idempotent
    assert np.array_equal(orc.s_soft(_bits(S)), S)
    # sign equivariance and positive homogeneity (power-of-two scale is exact)
    assert np.array_equal(orc.s_soft(_bits(-Wf)), -S + 0.0)
    assert np.array_equal(orc.s_soft(_bits(4 * Wf)), 4 * S)
    # permutation equivariance inside groups
    perm = [2, 0, 3, 1]
    Wp = Wf.reshape(-1, 4)[:, perm].reshape(Wf.shape)
    Sp = S.reshape(-1, 4)[:, perm].reshape(S.shape)
    assert np.array_equal(orc.s_soft(_bits(Wp)), Sp)


def test_s_soft_continuity_bound():
    """Proof of Theorem 4.1: a perturbation below delta moves every output by at most 2*delta."""
    rng = np.random.default_rng(3)
    base = np.round(np.clip(rng.standard_normal((4096, 4)), -1.9, 1.9) * 4) / 4   # many exact ties
    for delta in (2.0 ** -4, 2.0 ** -3):
        e = rng.integers(-4, 5, base.shape) * (delta / 4)                # bf16-exact perturbation
        A, B = base.astype(np.float32), (base + e).astype(np.float32)
        assert np.array_equal(synth.bf16_bits_to_f32(_bits(B)), B)
        SA, SB = orc.s_soft(_bits(A)), orc.s_soft(_bits(B))
        assert np.abs(SA.astype(np.float64) - SB).max() <= 2 * np.abs(e).max()
    # on a flip boundary (|t2| == |t3|) at least three outputs are zero
    tie = np.array([[0.5, 1.0, -1.0, 2.0]], np.float32)
    assert (orc.s_soft(_bits(tie)) != 0).sum() == 1


def test_beta_hand_worked_and_invariants():
    # groups [1,2,3,4] -> S_soft = [0,0,1,2]; <w,s> = 3 + 8 = 11, ||s||^2 = 5
    W = _bits(np.tile([1.0, 2.0, 3.0, 4.0], (8, 4)))
    b, num, den, deg = orc.beta(W)
    assert (b, deg) == (11.0 / 5.0, False)
    assert num / den == b
    # an already 2:4-sparse tensor is its own projection: beta = 1
    W = _bits(np.tile([0.0, 3.0, 0.0, -1.5], (4, 8)))
    assert orc.beta(W)[0] == 1.0
    # S_soft(w) == 0 (all magnitudes equal): degenerate, beta = 1
    b, _, den, deg = orc.beta(_bits(np.full((4, 16), 2.0)))
    assert (b, den, deg) == (1.0, 0.0, True)
    # scale invariance (power of two: exact) and beta >= 1
    W = synth.gaussian_bf16(7, (128, 256), 0.02)
    b1 = orc.beta(W)[0]
    b2 = orc.beta(_bits(synth.bf16_bits_to_f32(W) * 8))[0]
    assert b1 == b2 and b1 >= 1.0


def test_beta_minimises_mse():
    """Eq. 5: beta is the argmin over b of ||w - b S_soft(w)||^2."""
    W = synth.gaussian_bf16(9, (256, 256), 0.02)
    w = synth.bf16_bits_to_f32(W).astype(np.float64)
    A = w.reshape(-1, 4)
    t = np.sort(np.abs(A), axis=1)[:, 1:2]
    s = (np.sign(A) * np.maximum(np.abs(A) - t, 0)).reshape(w.shape)
    b = orc.beta(W)[0]
    mse = lambda x: ((w - x * s) ** 2).sum()
    assert mse(b) <= mse(b * (1 + 1e-4)) and mse(b) <= mse(b * (1 - 1e-4))
    # quadratic expansion of the MSE printed with Eq. 5
    assert np.isclose(mse(b), (w ** 2).sum() - 2 * b * (w * s).sum() + b * b * (s ** 2).sum(), rtol=1e-12)
    # i.i.d. Gaussian weights of any scale: beta ~ 1.48 (Monte-Carlo value, loose band)
    big = synth.gaussian_bf16(10, (2048, 2048), 0.02)
    assert abs(orc.beta(big)[0] - 1.4837) < 0.01


def test_compress_roundtrip_and_format():
    W = synth.gaussian_bf16(21, (128, 256), 0.02)
    Wf = synth.bf16_bits_to_f32(W)
    Wf[::3, ::5] = 0.0
    Wf[5] = 0.0
    Wf[7] = 0.25
    W = _bits(Wf)
    beta32 = np.float32(orc.beta(W)[0])
    vals, meta, dense = orc.project_compress(W, beta32)
    S = orc.s_soft(W)
    expect_dense = _bits(S * beta32)
    expect_dense[S == 0] = 0
    assert np.array_equal(dense, expect_dense)
    # decompress(compress) reproduces the dense projected tensor bit for bit
    back = orc.decompress(vals, meta)
    assert np.array_equal(_bits(back), dense)
    # every nibble is one of the six valid (p0 < p1) codes
    nibs = np.stack([(meta >> (4 * k)) & 0xF for k in range(4)], -1).reshape(-1)
    assert set(np.unique(nibs)) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    # every nonzero of S_soft sits at a kept position
    kept = orc.decompress(np.full_like(vals, 0x3F80), meta) != 0
    assert kept.reshape(-1, 4).sum(1).tolist() == [2] * (kept.size // 4)
    assert (kept | (S == 0)).all()
    # FP8 output: the same positions, values E4M3(fl32(fl32(s*beta)*scale))
    scale = np.float32(37.5)
    v8, m8, d8 = orc.project_compress(W, beta32, odt=orc.E4M3, wscale=scale)
    assert np.array_equal(m8, meta)
    import torch
    ref = (torch.from_numpy((S * beta32) * scale)).to(torch.float8_e4m3fn).view(torch.uint8).numpy().copy()
    ref[S == 0] = 0
    assert np.array_equal(d8, ref)
    assert np.array_equal(orc.f32_to_fp8(orc.decompress(v8, m8, orc.E4M3), orc.E4M3), d8)
