"""Pins for the oracle's casts, Philox stream, MVUE estimator (Sec. 5.1) and fp64 products.

Casts are checked against torch's CPU conversions (a library routine), Philox
against published known answers, MVUE against the properties its name fixes
(exactly 2:4, unbiased, variance equal to the closed-form lower bound, identity
on already-sparse groups, the textbook 1:2 special case) and the products
against triple loops and a library dense GEMM.
"""
import os

import numpy as np
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _bits(x):
    return synth.to_bf16_bits(np.asarray(x, np.float32))


# ------------------------------------------------------------------ casts

def test_bf16_codec_matches_torch():
    rng = np.random.default_rng(0)
    x = np.concatenate([
        (rng.standard_normal(100000) * 10.0 ** rng.integers(-30, 30, 100000)).astype(np.float32),
        np.array([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895314e38, 1e-40, -1e-45, np.inf, -np.inf],
                 np.float32),
        # exact ties between two bf16 neighbours: must go to even
        (np.arange(0x3F80, 0x3FA0, dtype=np.uint32) << 16 | 0x8000).view(np.float32),
    ])
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.f32_to_bf16(x), want)
    assert np.array_equal(synth.to_bf16_bits(x[np.isfinite(x)]), want[np.isfinite(x)])
    allbits = np.arange(65536, dtype=np.uint16)
    back = torch.from_numpy(allbits.view(np.int16)).view(torch.bfloat16).float().numpy()
    assert np.array_equal(orc.bf16_to_f32(allbits).view(np.uint32), back.view(np.uint32))


def test_fp8_decode_all_codes_match_torch():
    codes = np.arange(256, dtype=np.uint8)
    for dt, tdt in ((orc.E4M3, torch.float8_e4m3fn), (orc.E5M2, torch.float8_e5m2)):
        want = torch.from_numpy(codes).view(tdt).float().numpy()
        got = orc.fp8_to_f32(codes, dt)
        assert np.array_equal(np.isnan(got), np.isnan(want))
        ok = ~np.isnan(want)
        assert np.array_equal(got[ok].view(np.uint32), want[ok].view(np.uint32))


def test_fp8_encode_matches_torch_in_range_and_saturates():
    rng = np.random.default_rng(1)
    for dt, tdt, fmax in ((orc.E4M3, torch.float8_e4m3fn, 448.0), (orc.E5M2, torch.float8_e5m2, 57344.0)):
        codes = np.arange(256, dtype=np.uint8)
        vals = orc.fp8_to_f32(codes, dt)
        finite = vals[np.isfinite(vals)]
        pos = np.sort(finite[finite >= 0])
        mids = ((pos[:-1].astype(np.float64) + pos[1:]) / 2).astype(np.float32)   # exact ties
        x = np.concatenate([
            finite, mids, -mids, np.nextafter(mids, np.float32(0)), np.nextafter(mids, np.float32(1e9)),
            rng.uniform(-fmax, fmax, 200000).astype(np.float32),
            (rng.standard_normal(200000) * 2.0 ** rng.integers(-20, 8, 200000)).astype(np.float32),
        ])
        x = x[np.abs(x) <= fmax]
        want = torch.from_numpy(x).to(tdt).view(torch.uint8).numpy()
        assert np.array_equal(orc.f32_to_fp8(x, dt), want)
        # round trip of every finite code
        fin_codes = codes[np.isfinite(vals)]
        assert np.array_equal(orc.f32_to_fp8(orc.fp8_to_f32(fin_codes, dt), dt), fin_codes)
        # satfinite: beyond the largest finite value (and at infinity) the cast clamps
        top = orc.f32_to_fp8(np.array([fmax], np.float32), dt)[0]
        big = np.array([fmax * 1.5, 1e30, np.inf, -fmax * 2, -np.inf], np.float32)
        got = orc.f32_to_fp8(big, dt)
        assert got.tolist() == [top, top, top, top | 0x80, top | 0x80]
        assert orc.fp8_to_f32(np.array([top], np.uint8), dt)[0] == fmax


def test_amax_scale_quantize():
    X = synth.gaussian_bf16(3, (64, 128), 1.0)
    xf = synth.bf16_bits_to_f32(X)
    a = orc.amax(X)
    assert a == np.abs(xf).max()
    s = orc.fp8_scale(a, orc.E4M3)
    assert s == np.float32(448.0) / np.float32(a) and orc.fp8_scale(0.0, orc.E4M3) == 1.0
    q = orc.quantize(X, s, orc.E4M3)
    want = torch.from_numpy(xf * s).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    assert np.array_equal(q, want)
    assert np.abs(orc.fp8_to_f32(q, orc.E4M3)).max() == 448.0      # the largest element lands on FP8_MAX


# ----------------------------------------------------------------- Philox

def test_philox_known_answers():
    n = 0
    with open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            c, k, r = [[int(v, 16) for v in part.split()] for part in line.split("|")]
            assert orc.philox4x32_10(c, k).tolist() == r
            n += 1
    assert n == 3


# ------------------------------------------------------------------- MVUE

def _draws(a, n=10000):
    u = (np.arange(n, dtype=np.float64) + 0.5) / n          # stratified uniforms ...
    u = np.floor(u * 2 ** 24) / 2 ** 24                     # ... snapped to the generator's 2^-24 grid
    out = np.zeros((n, 4), np.float64)
    for k in range(n):
        pos, val = orc.mvue_group(a, np.float32(u[k]))
        assert pos[0] < pos[1]
        out[k, pos[0]] = val[0]
        out[k, pos[1]] = val[1]
    return out


def test_mvue_group_exactly_two_unbiased_min_variance():
    rng = np.random.default_rng(5)
    groups = [
        [0.5, -0.25, 0.125, 0.75],      # unclipped: 0.75 < 0.875
        [1.0, 1.0, 1.0, 1.0],           # all equal: two outputs of magnitude 2c
        [4.0, -0.5, 0.25, 1.0],         # clipped: 4 >= 1.75
        [0.0, 0.3, -0.2, 0.1],          # unclipped with a zero
        [1.0, 0.5, 0.25, 0.25],         # boundary m_x == rest (clipped branch, p_x = 1 either way)
    ] + rng.standard_normal((6, 4)).tolist()
    for a in groups:
        a = np.asarray(a, np.float32)
        m = np.abs(a.astype(np.float64))
        th = _draws(a, 4000)
        assert ((th != 0).sum(1) <= 2).all()
        # unbiased: systematic sampling over a stratified u grid integrates to a_i up to grid error
        assert np.allclose(th.mean(0), a, atol=2e-3 * m.sum()), (a, th.mean(0))
        # total variance equals the closed-form minimum (sum a_i^2 (1/p_i - 1) at the optimal p)
        x = int(np.argmax(m))
        rest = m.sum() - m[x]
        if m[x] >= rest:
            vmin = rest ** 2 - (m ** 2).sum() + m[x] ** 2
        else:
            vmin = m.sum() ** 2 / 2 - (m ** 2).sum()
        var = ((th - a.astype(np.float64)) ** 2).sum(1).mean()
        assert np.isclose(var, vmin, rtol=5e-3, atol=1e-6), (a, var, vmin)
        # any other unbiased 2-of-4 scheme is no better: uniform pairs, value 2*a_i
        var_uniform = (m ** 2).sum()            # sum a_i^2 (1/0.5 - 1)
        assert vmin <= var_uniform + 1e-12
    # all-equal group: both outputs are +-2c
    pos, val = orc.mvue_group(np.array([1, -1, 1, -1], np.float32), np.float32(0.3))
    assert sorted(np.abs(val).tolist()) == [2.0, 2.0]


def test_mvue_identity_on_sparse_groups_and_1of2_special_case():
    for a in ([0, 0, 5, -3], [0, 7, 0, 0], [0, 0, 0, 0], [2, 0, 0, -2], [-0.0, 3, 0, 1]):
        a = np.asarray(a, np.float32)
        for u in (0.0, 0.25, 0.5, 0.999):
            pos, val = orc.mvue_group(a, np.float32(u))
            out = np.zeros(4, np.float32)
            out[pos] = val
            assert np.array_equal(out, a + 0.0), (a, u, out)
    # [big, a1, a2, 0] with big >= a1+a2: the remaining slot is the textbook 1:2 estimator:
    # keep a1 with probability |a1|/(|a1|+|a2|), value sign*(|a1|+|a2|)
    a = np.array([8.0, 3.0, -1.0, 0.0], np.float32)
    th = _draws(a, 4000)
    assert (th[:, 0] == 8.0).all() and (th[:, 3] == 0).all()
    p1 = (th[:, 1] != 0).mean()
    assert abs(p1 - 0.75) < 1e-3
    assert set(np.unique(th[:, 1])) == {0.0, 4.0} and set(np.unique(th[:, 2])) == {0.0, -4.0}


def test_mvue_tensor_unbiased_over_philox_draws():
    """Sample mean over 10^4 Philox draws (steps 0..9999) converges to dY: |mean - a| <= 5 sigma/sqrt(n)."""
    T, O, n = 16, 8, 10000
    dY = synth.gaussian_bf16(77, (T, O), 1.0)
    a = synth.bf16_bits_to_f32(dY).astype(np.float64)
    acc = np.zeros((T, O))
    acc2 = np.zeros((T, O))
    for step in range(n):
        _, _, _, theta = orc.mvue(dY, seed=1234, tensor_id=3, step=step, want_theta=True)
        acc += theta
        acc2 += theta.astype(np.float64) ** 2
    mean = acc / n
    var = np.maximum(acc2 / n - mean ** 2, 0)
    assert (np.abs(mean - a) <= 5 * np.sqrt(var / n) + 1e-9).all()
    # Gaussian groups fall in the clipped case about one time in three (loose band)
    A = np.abs(synth.bf16_bits_to_f32(synth.gaussian_bf16(78, (4000, 4), 1.0)))
    frac = (A.max(1) >= A.sum(1) - A.max(1)).mean()
    assert 0.28 < frac < 0.39


def test_mvue_tensor_layout_counter_and_casts():
    T, O = 32, 12
    dY = synth.gaussian_bf16(79, (T, O), 1e-2)
    a = synth.bf16_bits_to_f32(dY)
    gvals, gmeta, _, theta = orc.mvue(dY, seed=(7 << 32) | 9, tensor_id=2, step=5, want_theta=True)
    assert gvals.shape == (O, T // 2) and gmeta.shape == (O, T // 16)
    # transposed canonical format decompresses to theta^T, values RNE bf16 of theta
    back = orc.decompress(gvals, gmeta)
    assert np.array_equal(_bits(back), _bits(theta.T.copy()))
    assert ((theta.reshape(T // 4, 4, O) != 0).sum(1) <= 2).all()
    # per-group recomputation from the documented counter mapping
    for tg, j in ((0, 0), (3, 5), (7, 11)):
        g = tg * O + j
        r = orc.philox4x32_10([g >> 2, 0, 2, 5], [9, 7])
        u = np.float32(int(r[g & 3]) >> 8) * np.float32(2.0 ** -24)
        pos, val = orc.mvue_group(a[4 * tg:4 * tg + 4, j], u)
        col = np.zeros(4, np.float32)
        col[pos] = val
        assert np.array_equal(col, theta[4 * tg:4 * tg + 4, j])
    # different step / tensor id / seed give different draws
    for kw in (dict(seed=(7 << 32) | 9, tensor_id=2, step=6), dict(seed=(7 << 32) | 9, tensor_id=3, step=5),
               dict(seed=(8 << 32) | 9, tensor_id=2, step=5)):
        assert not np.array_equal(orc.mvue(dY, **kw)[1], gmeta)
    # the counter is the global group index: a token-prefix shard reproduces the same rows
    half = orc.mvue(dY[:16].copy(), seed=(7 << 32) | 9, tensor_id=2, step=5, want_theta=True)[3]
    assert np.array_equal(half, theta[:16])
    # FP8 path: E5M2(fl32(v * gscale)), dense copy E5M2(fl32(dY * gscale))
    gs = np.float32(1000.0)
    v8, m8, dq, th8 = orc.mvue(dY, seed=(7 << 32) | 9, tensor_id=2, step=5, odt=orc.E5M2, gscale=gs,
                               want_dense_q=True, want_theta=True)
    assert np.array_equal(m8, gmeta) and np.array_equal(th8, theta)
    want_dq = torch.from_numpy(a * gs).to(torch.float8_e5m2).view(torch.uint8).numpy()
    assert np.array_equal(dq, want_dq)
    want_v = torch.from_numpy(theta.T.copy() * gs).to(torch.float8_e5m2).view(torch.uint8).numpy()
    got_v = orc.f32_to_fp8(orc.decompress(v8, m8, orc.E5M2), orc.E5M2)
    assert np.array_equal(got_v[theta.T != 0], want_v[theta.T != 0])


# --------------------------------------------------------------- products

def test_products_vs_triple_loop_and_dense_library():
    O, I, T = 8, 16, 16
    W = synth.gaussian_bf16(31, (O, I), 0.5)
    X = synth.gaussian_bf16(32, (T, I), 1.0)
    dY = synth.gaussian_bf16(33, (T, O), 1.0)
    beta32 = np.float32(orc.beta(W)[0])
    vals, meta, dense = orc.project_compress(W, beta32)
    wt = synth.bf16_bits_to_f32(dense).astype(np.float64)
    x = synth.bf16_bits_to_f32(X).astype(np.float64)
    g = synth.bf16_bits_to_f32(dY).astype(np.float64)
    Y = orc.linear_fwd(X, orc.BF16, vals, meta, orc.BF16)
    dX = orc.linear_bwd_input(dY, orc.BF16, dense, orc.BF16)
    gv, gm, _, theta = orc.mvue(dY, 1, 0, 0, want_theta=True)
    dW = orc.linear_bwd_weight(gv, gm, orc.BF16, X, orc.BF16)
    th = synth.bf16_bits_to_f32(_bits(theta)).astype(np.float64)
    for t in range(T):
        for o in range(O):
            assert np.isclose(Y[t, o], sum(x[t, i] * wt[o, i] for i in range(I)), rtol=1e-12, atol=1e-15)
        for i in range(I):
            assert np.isclose(dX[t, i], sum(g[t, o] * wt[o, i] for o in range(O)), rtol=1e-12, atol=1e-15)
    for o in range(O):
        for i in range(I):
            assert np.isclose(dW[o, i], sum(th[t, o] * x[t, i] for t in range(T)), rtol=1e-12, atol=1e-15)
    # W already 2:4 => beta = 1, S(W) = W and the forward is the library's dense product X W^T
    Wf = synth.bf16_bits_to_f32(synth.gaussian_bf16(34, (64, 128), 0.02)).reshape(64, 32, 4)
    Wf[:, :, [0, 2]] = 0
    W = _bits(Wf.reshape(64, 128))
    b = np.float32(orc.beta(W)[0])
    assert b == 1.0
    vals, meta, dense = orc.project_compress(W, b)
    assert np.array_equal(dense, W | 0) or np.array_equal(synth.bf16_bits_to_f32(dense), synth.bf16_bits_to_f32(W) + 0.0)
    X = synth.gaussian_bf16(35, (32, 128), 1.0)
    Y = orc.linear_fwd(X, orc.BF16, vals, meta, orc.BF16)
    lib = torch.from_numpy(synth.bf16_bits_to_f32(X)).double() @ torch.from_numpy(synth.bf16_bits_to_f32(W)).double().T
    assert np.allclose(Y, lib.numpy(), rtol=1e-12, atol=1e-15)
    # FP8: scales divide out
    sx, sw = np.float32(3.0), np.float32(5.0)
    Xq = orc.quantize(X, sx, orc.E4M3)
    v8, m8, _ = orc.project_compress(W, b, odt=orc.E4M3, wscale=sw)
    Y8 = orc.linear_fwd(Xq, orc.E4M3, v8, m8, orc.E4M3, inv_scale=1.0 / (float(sx) * float(sw)))
    assert np.linalg.norm(Y8 - Y) / np.linalg.norm(Y) < 0.08
