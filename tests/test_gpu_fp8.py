"""GPU parity of the FP8 whole-process variant (Sec. 5.2): E4M3 forward operands, E5M2 output gradient,
per-tensor scale = fp8_max / amax applied before the cast.  FP8 codes, metadata and scales must match the
oracle bit for bit; products within 5e-2 (relative Frobenius) of the fp64 product of the SAME quantised operands.
"""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, bits8, canonical_meta, dbf16, rel_fro

pytestmark = pytest.mark.gpu

FP8_GEMM_TOL = 5e-2


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def _f32(v):
    return torch.tensor([v], dtype=torch.float32, device=DEV)


def test_amax_scale_quantize(ctx):
    from paper_2409_09099_b200 import binding as B
    X = synth.bf16_bits_to_f32(synth.gaussian_bf16(1, (256, 384), 1.0))
    X[3, 5] = -64.0                                  # the maximum is negative
    X[0, :8] = [0.0, -0.0, 1e-30, 7.0, 1.0, -1.0, 3e-3, 2.0 ** -10]
    X = synth.to_bf16_bits(X)
    Xd = dbf16(X)
    amax = _f32(123.0)                               # stale content must not matter
    scale, inv = _f32(0), _f32(0)
    ctx.amax(Xd, amax)
    assert amax.item() == orc.amax(X) == 64.0
    for dt, tdt in ((B.E4M3, torch.float8_e4m3fn), (B.E5M2, torch.float8_e5m2)):
        ctx.fp8_scale(amax, dt, scale, inv)
        s_ref = orc.fp8_scale(64.0, dt)
        assert scale.item() == float(s_ref)
        assert inv.item() == float(np.float32(1.0) / s_ref)
        q = torch.empty(X.shape, dtype=tdt, device=DEV)
        ctx.quantize_fp8(Xd, amax, q)                # the kernel forms the scale from the amax itself
        assert np.array_equal(bits8(q), orc.quantize(X, s_ref, dt))
    zero = dbf16(np.zeros((128, 128), np.uint16))
    ctx.amax(zero, amax)
    ctx.fp8_scale(amax, B.E4M3, scale, inv)
    assert (amax.item(), scale.item(), inv.item()) == (0.0, 1.0, 1.0)
    q = torch.empty((128, 128), dtype=torch.float8_e4m3fn, device=DEV)
    ctx.quantize_fp8(zero, amax, q)                  # amax = 0: scale 1, all codes +0
    assert not bits8(q).any()


@pytest.mark.parametrize("O,I", [(256, 256), (384, 640)])
def test_project_compress_e4m3(ctx, O, I):
    from paper_2409_09099_b200 import binding as B
    W = synth.bf16_bits_to_f32(synth.gaussian_bf16(O + 3 * I, (O, I), 0.02))
    W[::5, ::3] = 0.0
    W[2] = 0.125
    W = synth.to_bf16_bits(W)
    beta32, w_amax = np.float32(1.4375), np.float32(0.078125)
    wscale = orc.fp8_scale(w_amax, orc.E4M3)                       # the scale the kernel forms from the amax
    vals, meta = ctx.alloc_compressed(O, I, B.E4M3)
    dense = torch.empty((O, I), dtype=torch.float8_e4m3fn, device=DEV)
    ctx.project_compress(dbf16(W), _f32(beta32), vals, meta, dense, w_amax_dev=_f32(w_amax))
    ov, om, od = orc.project_compress(W, beta32, odt=orc.E4M3, wscale=wscale)
    assert np.array_equal(bits8(vals), ov)
    assert np.array_equal(canonical_meta(ctx, meta, O, I, B.E4M3), om)
    assert np.array_equal(bits8(dense), od)
    dec = torch.empty_like(dense)
    ctx.decompress(vals, meta, dec)
    assert np.array_equal(bits8(dec), od)
    # saturation: a far too small amax (a huge scale) clamps to +-448 instead of producing NaN codes
    tiny = np.float32(448e-9)
    ctx.project_compress(dbf16(W), _f32(beta32), vals, meta, dense, w_amax_dev=_f32(tiny))
    assert np.array_equal(bits8(dense), orc.project_compress(W, beta32, odt=orc.E4M3, wscale=orc.fp8_scale(tiny, orc.E4M3))[2])
    assert not (bits8(dense) & 0x7F == 0x7F).any()


@pytest.mark.parametrize("T,O", [(512, 256), (1152, 384)])
def test_mvue_e5m2(ctx, T, O):
    from paper_2409_09099_b200 import binding as B
    dY = synth.bf16_bits_to_f32(synth.gaussian_bf16(T + O, (T, O), 1e-2))
    dY[::3, ::7] = 0.0
    dY = synth.to_bf16_bits(dY)
    gscale = orc.fp8_scale(orc.amax(dY), orc.E5M2)
    gvals, gmeta = ctx.alloc_compressed(O, T, B.E5M2)
    dq = torch.empty((T, O), dtype=torch.float8_e5m2, device=DEV)
    ctx.mvue_sparsify(dbf16(dY), 99, 4, 2, gvals, gmeta, dense_q_out=dq, g_amax_dev=_f32(orc.amax(dY)))
    ogv, ogm, odq, _ = orc.mvue(dY, 99, 4, 2, odt=orc.E5M2, gscale=gscale, want_dense_q=True)
    assert np.array_equal(bits8(gvals), ogv)
    assert np.array_equal(canonical_meta(ctx, gmeta, O, T, B.E5M2), ogm)
    assert np.array_equal(bits8(dq), odq)
    # the kept positions do not depend on the output type
    g16, m16 = ctx.alloc_compressed(O, T, B.BF16)
    ctx.mvue_sparsify(dbf16(dY), 99, 4, 2, g16, m16)
    assert np.array_equal(canonical_meta(ctx, m16, O, T, B.BF16), ogm)


@pytest.mark.parametrize("tile_width", [0, 128, 192, 224, 256])
@pytest.mark.parametrize("O,I,T", [(256, 256, 512), (384, 640, 1152), (128, 384, 128)])
def test_fp8_products(ctx, O, I, T, tile_width):
    """Each product against the fp64 product of the decoded FP8 operands, times 1/(scale_a * scale_b)."""
    from paper_2409_09099_b200 import binding as B
    W = synth.gaussian_bf16(O + 11, (O, I), 0.02)
    X = synth.gaussian_bf16(O + 12, (T, I), 1.0)
    dY = synth.gaussian_bf16(O + 13, (T, O), 1e-2)
    beta32 = np.float32(orc.beta(W)[0])
    _, _, wt16 = orc.project_compress(W, beta32)
    aw, ax, ag = _f32(orc.amax(wt16)), _f32(orc.amax(X)), _f32(orc.amax(dY))
    sw = orc.fp8_scale(orc.amax(wt16), orc.E4M3)
    sx = orc.fp8_scale(orc.amax(X), orc.E4M3)
    sg = orc.fp8_scale(orc.amax(dY), orc.E5M2)
    vals, meta = ctx.alloc_compressed(O, I, B.E4M3)
    dense = torch.empty((O, I), dtype=torch.float8_e4m3fn, device=DEV)
    ctx.project_compress(dbf16(W), _f32(beta32), vals, meta, dense, w_amax_dev=aw)
    Xq = torch.empty((T, I), dtype=torch.float8_e4m3fn, device=DEV)
    ctx.quantize_fp8(dbf16(X), ax, Xq)
    gvals, gmeta = ctx.alloc_compressed(O, T, B.E5M2)
    dYq = torch.empty((T, O), dtype=torch.float8_e5m2, device=DEV)
    ctx.mvue_sparsify(dbf16(dY), 5, 0, 0, gvals, gmeta, dense_q_out=dYq, g_amax_dev=ag)
    ctx.debug_force_tile_width(tile_width)
    inv_xw = np.float32(np.float32(1) / sx) * np.float32(np.float32(1) / sw)
    inv_gx = np.float32(np.float32(1) / sg) * np.float32(np.float32(1) / sx)
    inv_gw = np.float32(np.float32(1) / sg) * np.float32(np.float32(1) / sw)
    for odt, tol in ((torch.float32, 1e-4), (torch.bfloat16, FP8_GEMM_TOL)):
        Y = torch.empty((T, O), dtype=odt, device=DEV)
        dW = torch.empty((O, I), dtype=odt, device=DEV)
        dX = torch.empty((T, I), dtype=odt, device=DEV)
        ya = torch.full((1,), 1e9, device=DEV)
        ctx.linear_fwd(Xq, vals, meta, Y, x_amax_dev=ax, w_amax_dev=aw, y_amax_out_dev=ya)
        ctx.linear_bwd_weight(gvals, gmeta, Xq, dW, g_amax_dev=ag, x_amax_dev=ax)
        ctx.linear_bwd_input(dYq, dense, dX, g_amax_dev=ag, w_amax_dev=aw)
        dXc = torch.empty_like(dX)                   # the same product from the compressed E4M3 weight
        ctx.linear_bwd_input(dYq, None, dXc, g_amax_dev=ag, w_amax_dev=aw, vals=vals, meta=meta)
        torch.cuda.synchronize()
        assert torch.equal(dXc.view(torch.uint8), dX.view(torch.uint8))
        assert ya.item() == Y.float().abs().max().item()
        Y_ref = orc.linear_fwd(bits8(Xq), orc.E4M3, bits8(vals), canonical_meta(ctx, meta, O, I, B.E4M3), orc.E4M3,
                               inv_scale=float(inv_xw))
        dW_ref = orc.linear_bwd_weight(bits8(gvals), canonical_meta(ctx, gmeta, O, T, B.E5M2), orc.E5M2, bits8(Xq),
                                       orc.E4M3, inv_scale=float(inv_gx))
        dX_ref = orc.linear_bwd_input(bits8(dYq), orc.E5M2, bits8(dense), orc.E4M3, inv_scale=float(inv_gw))
        assert rel_fro(Y.float().cpu().numpy(), Y_ref) <= tol
        assert rel_fro(dW.float().cpu().numpy(), dW_ref) <= tol
        assert rel_fro(dX.float().cpu().numpy(), dX_ref) <= tol
    ctx.debug_force_tile_width(0)
    # reported, not gated: distance to the unquantised bf16 path
    Y16 = orc.linear_fwd(X, orc.BF16, *orc.project_compress(W, beta32)[:2], orc.BF16)
    assert rel_fro(Y_ref, Y16) < 0.1


def test_fp8_layer_end_to_end(ctx):
    """The SsteLinear bookkeeping in FP8 mode reproduces the oracle's scale chain and products."""
    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.layer import SsteLinear
    O, I, T = 256, 384, 512
    W, X, dY = synth.gaussian_bf16(71, (O, I), 0.02), synth.gaussian_bf16(72, (T, I), 1.0), synth.gaussian_bf16(73, (T, O), 1e-2)
    lin = SsteLinear(ctx, dbf16(W), T, tensor_id=3, seed=11, fp8=True, dense_copy=True)
    lin.init_beta()
    lin.prune()
    Y = lin.forward(dbf16(X))
    dX, dW = lin.backward(dbf16(dY), step=4)
    torch.cuda.synchronize()
    beta32 = np.float32(lin.beta.item())
    _, _, wt16 = orc.project_compress(W, beta32)
    sw, sx, sg = (orc.fp8_scale(orc.amax(wt16), orc.E4M3), orc.fp8_scale(orc.amax(X), orc.E4M3),
                  orc.fp8_scale(orc.amax(dY), orc.E5M2))
    assert lin.amax.cpu().numpy().tolist() == [orc.amax(X), orc.amax(wt16), orc.amax(dY)]
    ov, om, od = orc.project_compress(W, beta32, odt=orc.E4M3, wscale=sw)
    assert np.array_equal(bits8(lin.vals), ov) and np.array_equal(bits8(lin.w_dense), od)
    Xq = orc.quantize(X, sx, orc.E4M3)
    assert np.array_equal(bits8(lin.Xq), Xq)
    ogv, ogm, odq, _ = orc.mvue(dY, 11, 3, 4, odt=orc.E5M2, gscale=sg, want_dense_q=True)
    assert np.array_equal(bits8(lin.gvals), ogv) and np.array_equal(bits8(lin.dYq), odq)
    Y_ref = orc.linear_fwd(Xq, orc.E4M3, ov, om, orc.E4M3, inv_scale=1.0 / (float(sx) * float(sw)))
    dW_ref = orc.linear_bwd_weight(ogv, ogm, orc.E5M2, Xq, orc.E4M3, inv_scale=1.0 / (float(sg) * float(sx)))
    dX_ref = orc.linear_bwd_input(odq, orc.E5M2, od, orc.E4M3, inv_scale=1.0 / (float(sg) * float(sw)))
    assert rel_fro(Y.float().cpu().numpy(), Y_ref) <= FP8_GEMM_TOL
    assert rel_fro(dW.float().cpu().numpy(), dW_ref) <= FP8_GEMM_TOL
    assert rel_fro(dX.float().cpu().numpy(), dX_ref) <= FP8_GEMM_TOL


@pytest.mark.parametrize("O,I", [(128, 128), (384, 640), (1024, 4096)])
def test_project_amax_equals_amax_of_the_projection(ctx, O, I):
    """The read-only pass gives bit for bit the amax of the bf16 projection (oracle and GPU two-pass route)."""
    from paper_2409_09099_b200 import binding as B
    W = synth.gaussian_bf16(O * 3 + I, (O, I), 0.02)
    W[0, :4] = orc.f32_to_bf16(np.array([3.0, -2.5, 0.5, 0.25], dtype=np.float32))     # a clear maximum: (3 - 0.5) beta
    beta32 = np.float32(1.4837)
    beta = torch.full((1,), float(beta32), dtype=torch.float32, device=DEV)
    a1 = torch.full((1,), -1.0, dtype=torch.float32, device=DEV)
    for _ in range(2):                                           # the call zeroes its own accumulator
        ctx.project_amax(dbf16(W), beta, a1)
    vals, meta = ctx.alloc_compressed(O, I)
    dense = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
    ctx.project_compress(dbf16(W), beta, vals, meta, dense)
    a2 = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.amax(dense, a2)
    ref = orc.amax(orc.project_compress(W, beta32)[2])
    assert a1.item() == a2.item() == float(ref)
    zero = torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV)
    ctx.project_amax(zero, beta, a1)
    assert a1.item() == 0.0
