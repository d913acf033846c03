"""GPU parity: every libsste call, through the C ABI, against the CPU oracle on the same seeded inputs.

Bar: bit-exact for projected values, metadata, MVUE outputs and FP8 codes (given the same fp32
beta / scales); beta within 1e-6 relative; products within a relative Frobenius error of 1e-2
(bf16) / 5e-2 (FP8) of the fp64 product of the same operand bits.
"""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, bits8, canonical_meta, dbf16, rel_fro

pytestmark = pytest.mark.gpu

BF16_GEMM_TOL = 1e-2      # relative Frobenius error vs the fp64 product, bf16 operands and bf16 output
FP8_GEMM_TOL = 5e-2
BETA_TOL = 1e-6


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def _adversarial_weight(seed, O, I):
    """Gaussian weights with exact ties, zeros, an all-equal row and an all-zero row."""
    W = synth.bf16_bits_to_f32(synth.gaussian_bf16(seed, (O, I), 0.02))
    rng = np.random.default_rng(seed + 99)
    mask = rng.random(W.shape) < 0.15
    W[mask] = np.round(W[mask] * 128) / 128          # coarse grid: many ties inside groups
    W[::7, ::3] = 0.0
    W[3] = 0.25
    W[5] = 0.0
    W[6, ::2] = -0.0
    return synth.to_bf16_bits(W)


SHAPES = [(256, 256, 512), (384, 640, 1152), (128, 128, 128)]   # (O, I, T): config 1, a ragged multi-tile case, one tile


@pytest.mark.parametrize("O,I,T", SHAPES)
def test_beta_and_project_compress(ctx, O, I, T):
    from paper_2409_09099_b200 import binding as B
    W = _adversarial_weight(O + I, O, I)
    Wd = dbf16(W)
    beta_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(Wd, beta_dev)
    b_ref = orc.beta(W)[0]
    assert abs(beta_dev.item() - b_ref) <= BETA_TOL * abs(b_ref)
    # reproducible run to run (fixed reduction order)
    beta2 = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(Wd, beta2)
    assert beta2.item() == beta_dev.item()
    beta32 = np.float32(beta_dev.item())
    vals, meta = ctx.alloc_compressed(O, I)
    dense = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
    ctx.project_compress(Wd, beta_dev, vals, meta, dense)
    ov, om, od = orc.project_compress(W, beta32)
    assert np.array_equal(bits16(vals), ov)
    assert np.array_equal(canonical_meta(ctx, meta, O, I, B.BF16), om)
    assert np.array_equal(bits16(dense), od)
    # dense_out is optional
    vals2, meta2 = ctx.alloc_compressed(O, I)
    ctx.project_compress(Wd, beta_dev, vals2, meta2, None)
    assert torch.equal(vals2.view(torch.int16), vals.view(torch.int16)) and torch.equal(meta2, meta)


def test_beta_degenerate_and_sparse_input(ctx):
    O = I = 128
    beta_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(dbf16(synth.to_bf16_bits(np.full((O, I), 2.0, np.float32))), beta_dev)
    assert beta_dev.item() == 1.0
    assert ctx.poll_device_status() == 8          # SSTE_ERR_DEGENERATE recorded, then cleared
    assert ctx.poll_device_status() == 0
    W = synth.bf16_bits_to_f32(synth.gaussian_bf16(4, (O, I), 0.02)).reshape(O, I // 4, 4)
    W[:, :, [1, 2]] = 0
    ctx.beta_init(dbf16(synth.to_bf16_bits(W.reshape(O, I))), beta_dev)
    assert beta_dev.item() == 1.0 and ctx.poll_device_status() == 0


@pytest.mark.parametrize("O,I,T", SHAPES)
def test_mvue_sparsify(ctx, O, I, T):
    from paper_2409_09099_b200 import binding as B
    dY = synth.bf16_bits_to_f32(synth.gaussian_bf16(T + O, (T, O), 1e-2))
    dY[::5, ::3] = 0.0                      # groups with zeros
    dY[8:12, 7] = 0.0                       # an all-zero group
    dY[12:16, 9] = [0.0, 3.0, 0.0, 0.0]     # one nonzero
    dY[16:20, 11] = 0.5                     # all equal
    dY[20:24, 13] = [4.0, -0.5, 0.25, 1.0]  # clipped
    dY = synth.to_bf16_bits(dY)
    seed, tid, step = (0xABCD << 32) | 0x1234, 5, 17
    gvals, gmeta = ctx.alloc_compressed(O, T)
    ctx.mvue_sparsify(dbf16(dY), seed, tid, step, gvals, gmeta)
    ogv, ogm, _, _ = orc.mvue(dY, seed, tid, step)
    assert np.array_equal(bits16(gvals), ogv)
    assert np.array_equal(canonical_meta(ctx, gmeta, O, T, B.BF16), ogm)
    # another step draws other bits
    gvals2, gmeta2 = ctx.alloc_compressed(O, T)
    ctx.mvue_sparsify(dbf16(dY), seed, tid, step + 1, gvals2, gmeta2)
    assert not torch.equal(gmeta2, gmeta)
    assert np.array_equal(bits16(gvals2), orc.mvue(dY, seed, tid, step + 1)[0])
    # a data-parallel shard: the counter starts at the shard's first token, so the two halves of the
    # batch sparsified separately reproduce the unsharded result
    if T % 256 == 0:
        h = T // 2
        for t0 in (0, h):
            gv, gm = ctx.alloc_compressed(O, h)
            ctx.mvue_sparsify(dbf16(dY[t0:t0 + h].copy()), seed, tid, step, gv, gm, token_offset=t0)
            assert np.array_equal(bits16(gv), ogv[:, t0 // 2:(t0 + h) // 2])
            assert np.array_equal(bits16(gv), orc.mvue(dY[t0:t0 + h].copy(), seed, tid, step, token_offset=t0)[0])
    with pytest.raises(B.SsteError):
        ctx.mvue_sparsify(dbf16(dY), seed, tid, step, gvals, gmeta, token_offset=2)


@pytest.fixture(params=[0, 128, 192, 224, 256])
def tile_width(request, ctx):
    """Every tile-width variant of the product kernels (0 = the library's own choice)."""
    ctx.debug_force_tile_width(request.param)
    yield request.param
    ctx.debug_force_tile_width(0)


@pytest.mark.parametrize("O,I,T", SHAPES + [(768, 512, 1024)])
@pytest.mark.parametrize("out_dtype", [torch.bfloat16, torch.float32])
def test_three_products(ctx, O, I, T, out_dtype, tile_width):
    from paper_2409_09099_b200 import binding as B
    if out_dtype == torch.float32 and tile_width not in (0, 256):
        pytest.skip("fp32 output always uses 256-wide tiles")
    W, X, dY = _adversarial_weight(O, O, I), synth.gaussian_bf16(O + 1, (T, I), 1.0), synth.gaussian_bf16(O + 2, (T, O), 1e-2)
    Wd, Xd, dYd = dbf16(W), dbf16(X), dbf16(dY)
    beta_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(Wd, beta_dev)
    vals, meta = ctx.alloc_compressed(O, I)
    dense = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
    ctx.project_compress(Wd, beta_dev, vals, meta, dense)
    gvals, gmeta = ctx.alloc_compressed(O, T)
    ctx.mvue_sparsify(dYd, 7, 1, 0, gvals, gmeta)
    Y = torch.empty((T, O), dtype=out_dtype, device=DEV)
    dW = torch.empty((O, I), dtype=out_dtype, device=DEV)
    dX = torch.empty((T, I), dtype=out_dtype, device=DEV)
    ctx.linear_fwd(Xd, vals, meta, Y)
    ctx.linear_bwd_weight(gvals, gmeta, Xd, dW)
    ctx.linear_bwd_input(dYd, dense, dX)
    torch.cuda.synchronize()
    # the oracle multiplies the SAME operand bits (already verified bit-exact above) in fp64
    Y_ref = orc.linear_fwd(X, orc.BF16, bits16(vals), canonical_meta(ctx, meta, O, I, B.BF16), orc.BF16)
    dW_ref = orc.linear_bwd_weight(bits16(gvals), canonical_meta(ctx, gmeta, O, T, B.BF16), orc.BF16, X, orc.BF16)
    dX_ref = orc.linear_bwd_input(dY, orc.BF16, bits16(dense), orc.BF16)
    tol = BF16_GEMM_TOL if out_dtype == torch.bfloat16 else 1e-5
    assert rel_fro(Y.float().cpu().numpy(), Y_ref) <= tol
    assert rel_fro(dW.float().cpu().numpy(), dW_ref) <= tol
    assert rel_fro(dX.float().cpu().numpy(), dX_ref) <= tol
    # element-wise too: no entry is off by more than bf16 rounding of the accumulated value
    for got, ref in ((Y, Y_ref), (dW, dW_ref), (dX, dX_ref)):
        g = got.float().cpu().numpy().astype(np.float64)
        bound = 2.0 ** -7 * np.abs(ref) + 1e-4 * np.abs(ref).max()
        assert (np.abs(g - ref) <= bound).all()
    # grad_X from the COMPRESSED weight (expanded inside the product) is the same product bit for bit, and the
    # library's own decompression of the operand is the dense copy the projection wrote
    dX2 = torch.full_like(dX, 7.0)
    ctx.linear_bwd_input(dYd, None, dX2, vals=vals, meta=meta)
    assert torch.equal(dX2.view(torch.int32 if out_dtype == torch.float32 else torch.int16),
                       dX.view(torch.int32 if out_dtype == torch.float32 else torch.int16))
    dec = torch.empty_like(dense)
    ctx.decompress(vals, meta, dec)
    assert torch.equal(dec.view(torch.int16), dense.view(torch.int16))
    # optional amax outputs: max |Y|, max |grad_X| of the stored tensors (stale content must not matter)
    ya, xa = torch.full((1,), 1e9, device=DEV), torch.full((1,), 1e9, device=DEV)
    Y2 = torch.empty_like(Y)
    ctx.linear_fwd(Xd, vals, meta, Y2, y_amax_out_dev=ya)
    ctx.linear_bwd_input(dYd, None, dX2, vals=vals, meta=meta, dx_amax_out_dev=xa)
    assert torch.equal(Y2, Y)
    assert ya.item() == Y.float().abs().max().item() and xa.item() == dX.float().abs().max().item()
    if out_dtype == torch.bfloat16:
        assert ya.item() == orc.amax(bits16(Y)) and xa.item() == orc.amax(bits16(dX))


@pytest.mark.parametrize("splits", [1, 2, 3, 4])
@pytest.mark.parametrize("O,I,T", [(256, 3072, 3072), (2048, 256, 512)])
def test_split_k_products(ctx, O, I, T, splits):
    """Split-K (fp32 partial tiles in the workspace, summed in split order) gives the same products,
    bit for bit from run to run, for every split factor the shape allows."""
    from paper_2409_09099_b200 import binding as B
    W, X, dY = synth.gaussian_bf16(O + 5, (O, I), 0.02), synth.gaussian_bf16(O + 6, (T, I), 1.0), synth.gaussian_bf16(O + 7, (T, O), 1e-2)
    Wd, Xd, dYd = dbf16(W), dbf16(X), dbf16(dY)
    beta_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(Wd, beta_dev)
    vals, meta = ctx.alloc_compressed(O, I)
    dense = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
    ctx.project_compress(Wd, beta_dev, vals, meta, dense)
    gvals, gmeta = ctx.alloc_compressed(O, T)
    ctx.mvue_sparsify(dYd, 7, 1, 0, gvals, gmeta)
    outs = []
    ctx.debug_force_splits(splits)
    try:
        for rep in range(2):
            Y = torch.empty((T, O), dtype=torch.bfloat16, device=DEV)
            dW = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
            dX = torch.empty((T, I), dtype=torch.bfloat16, device=DEV)
            ctx.linear_fwd(Xd, vals, meta, Y)
            ctx.linear_bwd_weight(gvals, gmeta, Xd, dW)
            ctx.linear_bwd_input(dYd, dense, dX)
            dXc, xa = torch.empty_like(dX), torch.zeros(1, device=DEV)
            ctx.linear_bwd_input(dYd, None, dXc, vals=vals, meta=meta, dx_amax_out_dev=xa)   # compressed weight, amax out
            torch.cuda.synchronize()
            assert torch.equal(dXc.view(torch.int16), dX.view(torch.int16))
            assert xa.item() == dX.float().abs().max().item()
            outs.append((Y, dW, dX))
    finally:
        ctx.debug_force_splits(0)
    for a, b in zip(outs[0], outs[1]):
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    Y, dW, dX = outs[0]
    Y_ref = orc.linear_fwd(X, orc.BF16, bits16(vals), canonical_meta(ctx, meta, O, I, B.BF16), orc.BF16)
    dW_ref = orc.linear_bwd_weight(bits16(gvals), canonical_meta(ctx, gmeta, O, T, B.BF16), orc.BF16, X, orc.BF16)
    dX_ref = orc.linear_bwd_input(dY, orc.BF16, bits16(dense), orc.BF16)
    assert rel_fro(Y.float().cpu().numpy(), Y_ref) <= BF16_GEMM_TOL
    assert rel_fro(dW.float().cpu().numpy(), dW_ref) <= BF16_GEMM_TOL
    assert rel_fro(dX.float().cpu().numpy(), dX_ref) <= BF16_GEMM_TOL
    assert ctx.poll_device_status() == 0


def test_minimal_workspace_never_splits():
    """A context created with the minimal workspace has no room for partial tiles and still computes."""
    from paper_2409_09099_b200 import binding as B
    c = B.Context(0, minimal_workspace=True)
    O, I, T = 256, 256, 4096
    X = synth.gaussian_bf16(1, (T, I), 1.0)
    dY = synth.gaussian_bf16(2, (T, O), 1e-2)
    gvals, gmeta = c.alloc_compressed(O, T)
    c.mvue_sparsify(dbf16(dY), 1, 0, 0, gvals, gmeta)
    dW = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
    c.debug_force_splits(4)
    c.linear_bwd_weight(gvals, gmeta, dbf16(X), dW)
    c.debug_force_splits(0)
    ref = orc.linear_bwd_weight(bits16(gvals), canonical_meta(c, gmeta, O, T, B.BF16), orc.BF16, X, orc.BF16)
    assert rel_fro(dW.float().cpu().numpy(), ref) <= BF16_GEMM_TOL
    assert c.poll_device_status() == 0
    c.close()


def test_forward_of_already_sparse_weight_is_the_dense_product(ctx):
    """W already 2:4 => beta = 1, S(W) = W: the sparse forward equals the plain product X W^T."""
    O, I, T = 256, 512, 384
    W = synth.bf16_bits_to_f32(synth.gaussian_bf16(41, (O, I), 0.02)).reshape(O, I // 4, 4)
    W[:, :, [0, 3]] = 0
    W = synth.to_bf16_bits(W.reshape(O, I))
    X = synth.gaussian_bf16(42, (T, I), 1.0)
    beta_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(dbf16(W), beta_dev)
    assert beta_dev.item() == 1.0
    vals, meta = ctx.alloc_compressed(O, I)
    ctx.project_compress(dbf16(W), beta_dev, vals, meta, None)
    Y = torch.empty((T, O), dtype=torch.float32, device=DEV)
    ctx.linear_fwd(dbf16(X), vals, meta, Y)
    ref = synth.bf16_bits_to_f32(X).astype(np.float64) @ synth.bf16_bits_to_f32(W).astype(np.float64).T
    assert rel_fro(Y.cpu().numpy(), ref) <= 1e-5


def test_argument_validation_launches_nothing(ctx):
    from paper_2409_09099_b200 import binding as B
    W = torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV)
    beta = torch.ones(1, dtype=torch.float32, device=DEV)
    vals, meta = ctx.alloc_compressed(128, 128)
    with pytest.raises(B.SsteError) as e:
        ctx.project_compress(torch.zeros((128, 192), dtype=torch.bfloat16, device=DEV), beta, vals, meta)
    assert e.value.code == B.ERR_SHAPE
    with pytest.raises(B.SsteError) as e:      # misaligned output pointer
        ctx.project_compress(W, beta, vals.view(-1)[4:4 + 128 * 32].view(128, 32), meta)
    assert e.value.code in (B.ERR_ALIGN, B.ERR_SHAPE)
    with pytest.raises(B.SsteError) as e:      # E5M2 is not a forward operand type
        ctx.linear_fwd(torch.zeros((128, 128), dtype=torch.float8_e5m2, device=DEV),
                       torch.zeros((128, 64), dtype=torch.float8_e5m2, device=DEV), meta,
                       torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV))
    assert e.value.code == B.ERR_DTYPE
    assert ctx.lib.sste_beta_init(ctx.handle, None, 128, 128, 0, None, None) == B.ERR_INVALID_ARG
    assert ctx.poll_device_status() == 0


@pytest.mark.parametrize("fp8", [False, True])
def test_overlapped_backward_equals_serial(ctx, fp8):
    """grad_W on a side stream (own context, own split-K workspace) beside grad_X gives the same bits as the
    two calls back to back, also when both products split their reduction."""
    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.layer import SsteLinear
    O, I, T = 768, 3072, 2048
    W = dbf16(synth.gaussian_bf16(71, (O, I), 0.02))
    X = dbf16(synth.gaussian_bf16(72, (T, I), 1.0))
    dY = dbf16(synth.gaussian_bf16(73, (T, O), 1e-2))
    side_ctx, side = B.Context(0), torch.cuda.Stream()
    try:
        lin = SsteLinear(ctx, W, T, tensor_id=1, seed=9, fp8=fp8)
        lin.init_beta(); lin.prune(); lin.forward(X)
        lin.backward(dY, step=2)
        torch.cuda.synchronize()
        dW0, dX0 = lin.dW.clone(), lin.dX.clone()
        lin.dW.zero_(); lin.dX.zero_()
        for _ in range(3):
            lin.sparsify_grad(dY, 2)
            lin.grad_weight_and_input(dY, side_ctx, side)
        torch.cuda.synchronize()
        assert torch.equal(lin.dW.view(torch.int16), dW0.view(torch.int16))
        assert torch.equal(lin.dX.view(torch.int16), dX0.view(torch.int16))
        assert side_ctx.poll_device_status() == 0
    finally:
        side_ctx.close()


@pytest.mark.parametrize("group_m", [1, 2, 3, 1000])
def test_tile_order_does_not_change_the_products(ctx, group_m):
    """Every band height of the tile order (incl. a last, partial band and split tail tiles) gives the same bits."""
    O, I, T = 1280, 768, 1792                      # forward 5 x 7, grad_W 5 x 3, grad_X 7 x 3 tiles of 256 x 256
    W, X, dY = synth.gaussian_bf16(91, (O, I), 0.02), synth.gaussian_bf16(92, (T, I), 1.0), synth.gaussian_bf16(93, (T, O), 1e-2)
    Wd, Xd, dYd = dbf16(W), dbf16(X), dbf16(dY)
    beta_dev = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(Wd, beta_dev)
    vals, meta = ctx.alloc_compressed(O, I)
    dense = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
    ctx.project_compress(Wd, beta_dev, vals, meta, dense)
    gvals, gmeta = ctx.alloc_compressed(O, T)
    ctx.mvue_sparsify(dYd, 7, 1, 0, gvals, gmeta)

    def run():
        Y = torch.empty((T, O), dtype=torch.bfloat16, device=DEV)
        dW = torch.empty((O, I), dtype=torch.bfloat16, device=DEV)
        dX = torch.empty((T, I), dtype=torch.bfloat16, device=DEV)
        dXc = torch.empty((T, I), dtype=torch.bfloat16, device=DEV)
        ctx.linear_fwd(Xd, vals, meta, Y)
        ctx.linear_bwd_weight(gvals, gmeta, Xd, dW)
        ctx.linear_bwd_input(dYd, dense, dX)
        ctx.linear_bwd_input(dYd, None, dXc, vals=vals, meta=meta)
        torch.cuda.synchronize()
        return Y, dW, dX, dXc

    # the same split plan on both sides: the order of the tiles must not change a single bit
    results = {}
    try:
        for splits in (1, 2):
            ctx.debug_force_splits(splits)
            for order in (1000, group_m):
                ctx.debug_force_tile_order(order)
                results[splits, order] = run()
    finally:
        ctx.debug_force_splits(0)
        ctx.debug_force_tile_order(0)
    for splits in (1, 2):
        for a, b in zip(results[splits, 1000], results[splits, group_m]):
            assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    refs = (orc.linear_fwd(X, orc.BF16, bits16(vals), canonical_meta(ctx, meta, O, I, 0), orc.BF16),
            orc.linear_bwd_weight(bits16(gvals), canonical_meta(ctx, gmeta, O, T, 0), orc.BF16, X, orc.BF16),
            orc.linear_bwd_input(dY, orc.BF16, bits16(dense), orc.BF16))
    for a, ref in zip(results[2, group_m][:3], refs):
        assert rel_fro(a.float().cpu().numpy(), ref) <= BF16_GEMM_TOL
    assert ctx.poll_device_status() == 0


@pytest.mark.parametrize("fp8", [False, True])
def test_projection_on_every_group_over_an_alphabet(ctx, fp8):
    """All 12^4 groups over an alphabet with zeros, -0, subnormals, adjacent bf16 values, ties and huge ratios:
    values, metadata and dense copy bit for bit (bf16 and E4M3), and the beta reduction on the same tensor."""
    from paper_2409_09099_b200 import binding as B
    alphabet = np.array([0.0, -0.0, 1.0, -1.0, 1.0078125, 2.0, -3.0, 0.5, 2.0 ** -17, 2.0 ** -126, -(2.0 ** -133), 65280.0],
                        dtype=np.float32)
    idx = np.stack(np.meshgrid(*[np.arange(len(alphabet))] * 4, indexing="ij"), -1).reshape(-1, 4)
    flat = np.zeros(128 * 768, np.float32)
    flat[: idx.size] = alphabet[idx].reshape(-1)
    W = synth.to_bf16_bits(flat.reshape(128, 768))
    O, I = W.shape
    beta32, w_amax = np.float32(1.4837), np.float32(65280.0 * 1.4837)
    dt, odt = (B.E4M3, orc.E4M3) if fp8 else (B.BF16, orc.BF16)
    vals, meta = ctx.alloc_compressed(O, I, dt)
    dense = torch.empty((O, I), dtype=B._TORCH_DT[dt], device=DEV)
    beta = torch.full((1,), float(beta32), dtype=torch.float32, device=DEV)
    amax = torch.full((1,), float(w_amax), dtype=torch.float32, device=DEV)
    ctx.project_compress(dbf16(W), beta, vals, meta, dense, w_amax_dev=amax if fp8 else None)
    ov, om, od = orc.project_compress(W, beta32, odt=odt, wscale=orc.fp8_scale(w_amax, orc.E4M3) if fp8 else 1.0)
    bits = (lambda t: t.view(torch.uint8).cpu().numpy()) if fp8 else bits16
    assert np.array_equal(bits(vals), ov)
    assert np.array_equal(bits(dense), od)
    assert np.array_equal(canonical_meta(ctx, meta, O, I, dt), om)
    got = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init(dbf16(W), got)
    ref = orc.beta(W)[0]
    assert abs(got.item() - ref) <= 1e-6 * abs(ref)
