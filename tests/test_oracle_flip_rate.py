"""Pins of the oracle's flip rate r_k = ||m_h(w_k) xor m_h(w_{k-1})||_1 / d (Sec. 3.1, "Flip rate")."""
import itertools

import numpy as np

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth


def _bf16(x):
    return orc.f32_to_bf16(np.asarray(x, dtype=np.float32))


def test_hard_mask_by_brute_force_on_all_small_patterns():
    """Every group over a small alphabet: the mask keeps exactly the two elements ranked first by
    (magnitude descending, index ascending), found here by explicit ranking."""
    vals = [-2.0, -1.0, 0.0, 1.0, 3.0]
    groups = np.array(list(itertools.product(vals, repeat=4)), dtype=np.float32)
    mask = orc.hard_mask(_bf16(groups))
    for a, m in zip(groups, mask):
        rank = sorted(range(4), key=lambda i: (-abs(a[i]), i))
        want = np.zeros(4, dtype=np.uint8)
        want[rank[:2]] = 1
        assert np.array_equal(m, want)
        assert m.sum() == 2


def test_mask_is_the_kept_pattern_of_the_projection():
    """m_h is the pattern of the 2:4 metadata the projection emits (S_soft prunes the two smallest magnitudes)."""
    W = synth.gaussian_bf16(7, (64, 256), 0.02)
    _, meta, _ = orc.project_compress(W, np.float32(1.25))
    mask = orc.hard_mask(W).reshape(64, 64, 4)
    nib = np.stack([(meta >> (4 * j)) & 0xF for j in range(4)], axis=-1).reshape(64, 64)   # one nibble per group
    p0, p1 = nib & 3, nib >> 2
    want = np.zeros_like(mask)
    np.put_along_axis(want, p0[..., None].astype(np.int64), 1, axis=-1)
    np.put_along_axis(want, p1[..., None].astype(np.int64), 1, axis=-1)
    assert np.array_equal(mask, want)


def test_closed_forms():
    W = synth.gaussian_bf16(3, (32, 128), 0.02)
    assert orc.flip_count(W, W) == 0 and orc.flip_rate(W, W) == 0.0
    # scaling by a positive constant or flipping signs changes no magnitude order
    f = orc.bf16_to_f32(W)
    assert orc.flip_count(W, _bf16(-2.0 * f)) == 0
    # one group whose 2nd and 3rd magnitudes swap: exactly two mask entries change, rate 2 / d
    a = np.array([[4.0, 3.0, 2.0, 1.0]], dtype=np.float32)
    b = np.array([[4.0, 2.0, 3.0, 1.0]], dtype=np.float32)
    assert orc.flip_count(_bf16(a), _bf16(b)) == 2
    assert orc.flip_rate(_bf16(a), _bf16(b)) == 0.5
    # both kept entries replaced: four changes, the maximum for a group
    c = np.array([[1.0, 2.0, 4.0, 3.0]], dtype=np.float32)
    assert orc.flip_count(_bf16(a), _bf16(c)) == 4


def test_every_group_contributes_an_even_number_of_flips():
    """Both masks hold exactly two ones per group, so their XOR has 0, 2 or 4."""
    A = synth.gaussian_bf16(11, (16, 512), 0.02)
    B = synth.gaussian_bf16(12, (16, 512), 0.02)
    x = (orc.hard_mask(A) != orc.hard_mask(B)).reshape(16, 128, 4).sum(-1)
    assert set(np.unique(x)) <= {0, 2, 4}
    # independent tensors: two uniform 2-subsets of 4 coincide with probability 1/6, share one element with 4/6
    # and are disjoint with 1/6 -- 2 flips per group on average, rate 0.5
    rate = orc.flip_rate(A, B)
    assert abs(rate - 0.5) < 0.02


def test_small_perturbation_flips_few():
    W = synth.gaussian_bf16(5, (64, 512), 0.02)
    f = orc.bf16_to_f32(W)
    rng = np.random.default_rng(0)
    W2 = _bf16(f + 1e-4 * rng.standard_normal(f.shape).astype(np.float32))
    r = orc.flip_rate(W, W2)
    assert 0.0 < r < 0.05
