"""GPU parity on seeded random shapes (multiples of 128, ragged against every tile size) with adversarial
content, through the whole layer: elementwise outputs bit for bit, the three products against fp64."""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, bits8, canonical_meta, dbf16, rel_fro

pytestmark = pytest.mark.gpu

_RNG = np.random.default_rng(20240913)
_SHAPES = [tuple(int(128 * _RNG.integers(1, 13)) for _ in range(3)) for _ in range(10)]


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def _adversarial(a, rng):
    g = a.reshape(-1, 4)
    idx = rng.choice(g.shape[0], size=max(1, g.shape[0] // 8), replace=False)
    g[idx[0::4], 1] = g[idx[0::4], 2]          # ties
    g[idx[1::4], :] = g[idx[1::4], :1]         # all-equal groups
    g[idx[2::4], :] = 0                        # zero groups
    g[idx[3::4], 0] = 0x8000                   # -0
    return a


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("O,I,T", _SHAPES)
def test_layer_on_random_shape(ctx, O, I, T, fp8):
    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.layer import SsteLinear
    rng = np.random.default_rng(O * 7 + I * 3 + T)
    W = _adversarial(synth.gaussian_bf16(O + 1, (O, I), 0.02), rng)
    X = synth.gaussian_bf16(I + 2, (T, I), 1.0)
    # groups of the gradient run along tokens: adversarial structure on the transposed view
    dY = np.ascontiguousarray(_adversarial(np.ascontiguousarray(synth.gaussian_bf16(T + 3, (T, O), 1e-2).T), rng).T)
    # half of the shapes keep a dense copy of w~ for grad_X, the others expand the compressed operand in the product
    lin = SsteLinear(ctx, dbf16(W), T, tensor_id=5, seed=77, fp8=fp8, dense_copy=bool((O // 128) & 1))
    dec = torch.empty((O, I), dtype=lin.vals.dtype, device=DEV)
    lin.init_beta(); lin.prune(); lin.forward(dbf16(X)); lin.backward(dbf16(dY), step=11)
    torch.cuda.synchronize()
    beta32 = np.float32(lin.beta.item())
    assert abs(float(beta32) - orc.beta(W)[0]) <= 1e-6 * float(beta32)
    if not fp8:
        ov, om, od = orc.project_compress(W, beta32)
        ogv, ogm, _, _ = orc.mvue(dY, 77, 5, 11)
        ctx.decompress(lin.vals, lin.meta, dec)
        assert np.array_equal(bits16(lin.vals), ov) and np.array_equal(bits16(dec), od)
        assert lin.w_dense is None or np.array_equal(bits16(lin.w_dense), od)
        assert np.array_equal(canonical_meta(ctx, lin.meta, O, I, B.BF16), om)
        assert np.array_equal(bits16(lin.gvals), ogv)
        assert np.array_equal(canonical_meta(ctx, lin.gmeta, O, T, B.BF16), ogm)
        refs = (orc.linear_fwd(X, orc.BF16, ov, om, orc.BF16), orc.linear_bwd_weight(ogv, ogm, orc.BF16, X, orc.BF16),
                orc.linear_bwd_input(dY, orc.BF16, od, orc.BF16))
        tol = 1e-2
    else:
        _, _, wt16 = orc.project_compress(W, beta32)
        sw, sx, sg = (orc.fp8_scale(orc.amax(wt16), orc.E4M3), orc.fp8_scale(orc.amax(X), orc.E4M3),
                      orc.fp8_scale(orc.amax(dY), orc.E5M2))
        ov, om, od = orc.project_compress(W, beta32, odt=orc.E4M3, wscale=sw)
        Xq = orc.quantize(X, sx, orc.E4M3)
        ogv, ogm, odq, _ = orc.mvue(dY, 77, 5, 11, odt=orc.E5M2, gscale=sg, want_dense_q=True)
        ctx.decompress(lin.vals, lin.meta, dec)
        assert np.array_equal(bits8(lin.vals), ov) and np.array_equal(bits8(dec), od)
        assert lin.w_dense is None or np.array_equal(bits8(lin.w_dense), od)
        assert np.array_equal(canonical_meta(ctx, lin.meta, O, I, B.E4M3), om)
        assert np.array_equal(bits8(lin.gvals), ogv) and np.array_equal(bits8(lin.dYq), odq)
        assert np.array_equal(canonical_meta(ctx, lin.gmeta, O, T, B.E5M2), ogm)
        refs = (orc.linear_fwd(Xq, orc.E4M3, ov, om, orc.E4M3, 1.0 / (float(sx) * float(sw))),
                orc.linear_bwd_weight(ogv, ogm, orc.E5M2, Xq, orc.E4M3, 1.0 / (float(sg) * float(sx))),
                orc.linear_bwd_input(odq, orc.E5M2, od, orc.E4M3, 1.0 / (float(sg) * float(sw))))
        tol = 5e-2
    for got, ref in zip((lin.Y, lin.dW, lin.dX), refs):
        assert rel_fro(got.float().cpu().numpy(), ref) <= tol
