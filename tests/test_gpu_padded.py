"""Shapes that are not multiples of 128, run on zero-padded copies (sste_pad_2d / sste_crop_2d, SsteLinearPadded).

A group of four zeros is a fixed point of the projection (Eq. 4) and of the MVUE rule and adds nothing to beta
(Eq. 5) or to a product, so the padded run must reproduce the oracle on the UNPADDED tensors: projection, metadata
and MVUE bit for bit on the real rows and columns (the MVUE counter runs over the unpadded column count), products
within the bf16 tolerance.  The oracle wants whole 16-element metadata words along a group dimension, so a token
count that is not a multiple of 16 is zero-extended to the next one for it (those extra groups are zero groups).
Covers a vocabulary-sized projection (50257 rows: an odd column count for the MVUE counter) and small odd shapes.
"""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, canonical_meta, dbf16, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def test_pad_and_crop_round_trip(ctx):
    from paper_2409_09099_b200 import binding as B
    assert [B.padded_dim(n) for n in (1, 127, 128, 129, 50257)] == [128, 128, 128, 256, 50304]
    a = synth.gaussian_bf16(3, (203, 77), 1.0)
    src = dbf16(a)
    dst = torch.full((256, 128), 7.0, dtype=torch.bfloat16, device=DEV)
    ctx.pad_2d(src, dst)
    want = np.zeros((256, 128), np.uint16)
    want[:203, :77] = a
    assert np.array_equal(bits16(dst), want)
    back = torch.empty((203, 77), dtype=torch.bfloat16, device=DEV)
    ctx.crop_2d(dst, back)
    assert np.array_equal(bits16(back), a)
    lib = B.load()
    assert lib.sste_pad_2d(ctx.handle, None, 1, 1, None, 1, 8, None) == B.ERR_INVALID_ARG
    assert lib.sste_pad_2d(ctx.handle, src.data_ptr(), 203, 77, dst.data_ptr(), 128, 128, None) == B.ERR_SHAPE   # rows_p < rows
    assert lib.sste_pad_2d(ctx.handle, src.data_ptr(), 203, 77, dst.data_ptr(), 256, 100, None) == B.ERR_SHAPE   # cols_p % 8


@pytest.mark.parametrize("O,I,T", [(200, 208, 1000), (203, 80, 72), (50257, 768, 1024)])
def test_padded_layer_matches_the_unpadded_oracle(ctx, O, I, T):
    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.layer import SsteLinearPadded
    W = synth.gaussian_bf16(O + 1, (O, I), 0.02)
    X = synth.gaussian_bf16(O + 2, (T, I), 1.0)
    dY = synth.gaussian_bf16(O + 3, (T, O), 1e-2)
    lin = SsteLinearPadded(ctx, O, I, T, tensor_id=9, seed=21)
    lin.set_weight(dbf16(W))
    lin.init_beta()
    lin.prune()
    Y = lin.forward(dbf16(X))
    dX, dW = lin.backward(dbf16(dY), step=6)
    torch.cuda.synchronize()
    Op, Ip, Tp = lin.Op, lin.Ip, lin.Tp
    beta_ref = orc.beta(W)[0]
    assert abs(lin.beta.item() - beta_ref) <= 1e-6 * beta_ref
    # projection: real rows / columns equal the oracle's, the padding is zero groups kept at positions (0, 1)
    ov, om, od = orc.project_compress(W, np.float32(lin.beta.item()))
    inner = lin.inner
    assert np.array_equal(bits16(inner.vals)[:O, : I // 2], ov)
    assert not bits16(inner.vals)[O:].any() and not bits16(inner.vals)[:, I // 2:].any()
    gm = canonical_meta(ctx, inner.meta, Op, Ip, B.BF16)
    assert np.array_equal(gm[:O, : I // 16], om)
    assert (gm[O:] == 0x4444).all() and (gm[:, I // 16:] == 0x4444).all()
    # MVUE: the draws are those of the unpadded [T, O] gradient
    T16 = (T + 15) // 16 * 16
    dY16 = np.zeros((T16, O), np.uint16)
    dY16[:T] = dY
    X16 = np.zeros((T16, I), np.uint16)
    X16[:T] = X
    ogv, ogm, _, _ = orc.mvue(dY16, 21, 9, 6)
    gv = bits16(inner.gvals)
    assert np.array_equal(gv[:O, : T16 // 2], ogv)
    assert not gv[O:].any() and not gv[:, T16 // 2:].any()
    ggm = canonical_meta(ctx, inner.gmeta, Op, Tp, B.BF16)
    assert np.array_equal(ggm[:O, : T16 // 16], ogm)
    # products on the real region
    refs = (orc.linear_fwd(X, orc.BF16, ov, om, orc.BF16),
            orc.linear_bwd_weight(ogv, ogm, orc.BF16, X16, orc.BF16),
            orc.linear_bwd_input(dY, orc.BF16, od, orc.BF16))
    for got, ref in zip((Y, dW, dX), refs):
        assert tuple(got.shape) == ref.shape
        assert rel_fro(got.float().cpu().numpy(), ref) <= 1e-2
