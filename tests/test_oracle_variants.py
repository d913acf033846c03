"""Pins of the oracle's ablation variants of the pruning step (gamma threshold, hard threshold, L1 beta, SR-STE)."""
import numpy as np

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth


def _bf16(x):
    return orc.f32_to_bf16(np.asarray(x, dtype=np.float32))


def _f(x):
    return orc.bf16_to_f32(x)


def test_gamma_zero_is_the_default_projection():
    """gamma = 0 must reproduce the pinned C path bit for bit (bf16 and E4M3)."""
    W = synth.gaussian_bf16(2, (64, 256), 0.02)
    W[:4].reshape(-1, 4)[:, 1] = W[:4].reshape(-1, 4)[:, 2]          # ties
    W[4:6] = 0
    b = np.float32(1.4837)
    for odt, ws in ((orc.BF16, 1.0), (orc.E4M3, 37.5)):
        ref = orc.project_compress(W, b, odt=odt, wscale=ws)
        got = orc.project_compress_variant(W, b, gamma=0.0, odt=odt, wscale=ws)
        for r, g in zip(ref, got):
            assert np.array_equal(r, g)


def test_gamma_threshold_closed_forms():
    # sorted magnitudes 1, 2, 4, 8: t = (1-g)*2 + g*4
    a = _bf16([[8.0, -1.0, 4.0, -2.0] * 4])                           # four copies: one metadata word
    for g, t in ((0.0, 2.0), (0.25, 2.5), (0.5, 3.0), (1.0, 4.0)):
        _, meta, dense = orc.project_compress_variant(a, np.float32(1.0), gamma=g)
        want = np.array([[8.0 - t, 0.0, max(4.0 - t, 0.0), 0.0] * 4], dtype=np.float32)
        assert np.array_equal(_f(dense), want)
        assert int(meta[0, 0]) == 0x8888                              # kept positions stay the two largest: 0 | 2 << 2
    # the threshold stays feasible for every gamma in [0, 1]: at most two non-zeros, the two smallest are zero
    W = synth.gaussian_bf16(9, (32, 128), 0.02)
    for g in (0.0, 0.3, 0.7, 1.0):
        _, _, dense = orc.project_compress_variant(W, np.float32(1.0), gamma=g)
        nz = (_f(dense).reshape(-1, 4) != 0).sum(-1)
        assert nz.max() <= 2
        assert np.array_equal((_f(dense) != 0) & (orc.hard_mask(W) == 0), np.zeros(W.shape, dtype=bool))
    # a larger gamma shrinks the projection (Sec. 4.1)
    n = [np.abs(_f(orc.project_compress_variant(W, np.float32(1.0), gamma=g)[2])).sum() for g in (0.0, 0.5, 1.0)]
    assert n[0] > n[1] > n[2]


def test_hard_threshold_is_masking():
    W = synth.gaussian_bf16(4, (32, 128), 0.02)
    vals, meta, dense = orc.project_compress_variant(W, np.float32(1.0), hard=True)
    assert np.array_equal(_f(dense), _f(W) * orc.hard_mask(W))          # S_h(a) = a * m_h(a)  (Eq. 2)
    assert np.array_equal(orc.decompress(vals, meta), _f(dense))
    # same mask as the soft projection, larger magnitudes
    _, meta_s, dense_s = orc.project_compress(W, np.float32(1.0))
    assert np.array_equal(meta, meta_s)
    assert (np.abs(_f(dense)) >= np.abs(_f(dense_s))).all()
    # idempotent: a 2:4 tensor is its own hard projection
    _, _, again = orc.project_compress_variant(dense, np.float32(1.0), hard=True)
    assert np.array_equal(again, dense)


def test_beta_l1():
    a = _bf16([[4.0, -3.0, 2.0, 1.0]])                                # S_soft = (2, -1, 0, 0): 10 / 3
    assert abs(orc.beta_l1(a) - 10.0 / 3.0) < 1e-12
    W = synth.gaussian_bf16(6, (64, 256), 0.02)
    b1, b2 = orc.beta_l1(W), orc.beta(W)[0]
    s = orc.s_soft(W).astype(np.float64)
    assert abs(b1 * np.abs(s).sum() - np.abs(_f(W).astype(np.float64)).sum()) < 1e-9      # keeps the L1 norm
    assert b1 > b2 > 1.0                                              # keeping the magnitude overshoots the MSE optimum
    assert orc.beta_l1(_bf16(np.zeros((4, 16)))) == 1.0


def test_srste_decay():
    W = synth.gaussian_bf16(8, (16, 64), 0.02)
    dW = synth.gaussian_bf16(9, (16, 64), 1e-3)
    out = orc.srste_decay(dW, W, 0.5)
    kept = orc.hard_mask(W) == 1
    assert np.array_equal(out[kept], dW[kept])                        # kept weights feel no decay
    want = (_f(dW) + np.float32(0.5) * _f(W)).astype(np.float32)
    assert np.array_equal(out[~kept], _bf16(want)[~kept])
    assert np.array_equal(orc.srste_decay(dW, W, 0.0), dW)
    # the term is the gradient of (lambda / 2) ||w (1 - m)||^2: finite difference on one pruned entry
    w = _f(W).astype(np.float64)
    m = orc.hard_mask(W)
    i, j = np.argwhere(m == 0)[0]
    reg = lambda x: 0.25 * ((x * (1 - m)) ** 2).sum()
    e = np.zeros_like(w); e[i, j] = 1e-6
    assert abs((reg(w + e) - reg(w - e)) / 2e-6 - 0.5 * w[i, j]) < 1e-8
