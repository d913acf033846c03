"""GPU parity at the benchmark's full sizes, in the launch configuration bench.py times (SsteLinear call order,
library-chosen tile widths and split-K).

Config 2 (GPT-2-small MLP): everything compared in full -- projection, metadata, MVUE bit for bit, the three
products against complete fp64 products.  Every layer of config 3 (GPT-2-large block linears), the attention
linears of config 4 and every layer of config 5 (7B-shaped FFN, FP8): the elementwise outputs in full, the
products on a seeded sample of 256 output rows each, computed one by one as fp64 dot products of the decoded
operands.
"""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, bits8, canonical_meta, dbf16, rel_fro

pytestmark = pytest.mark.gpu

BF16_GEMM_TOL = 1e-2
FP8_GEMM_TOL = 5e-2
N_SAMPLE = 256


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def _run_layer(ctx, W, X, dY, tensor_id, seed, step, fp8):
    """The layer as bench.py runs it (library defaults)."""
    from paper_2409_09099_b200.layer import SsteLinear
    lin = SsteLinear(ctx, dbf16(W), X.shape[0], tensor_id=tensor_id, seed=seed, fp8=fp8)
    lin.init_beta()
    lin.prune()
    lin.forward(dbf16(X))
    lin.backward(dbf16(dY), step=step)
    torch.cuda.synchronize()
    return lin


@pytest.mark.parametrize("layer", [0, 1])
def test_config2_full(ctx, layer):
    from paper_2409_09099_b200 import binding as B
    cfg = synth.CONFIGS[2]
    W, X, dY = synth.layer_tensors(2, layer)
    O, I = W.shape
    T = X.shape[0]
    lin = _run_layer(ctx, W, X, dY, layer, cfg["seed"], 3, False)
    beta_ref = orc.beta(W)[0]
    assert abs(lin.beta.item() - beta_ref) <= 1e-6 * beta_ref
    ov, om, od = orc.project_compress(W, np.float32(lin.beta.item()))
    assert np.array_equal(bits16(lin.vals), ov) and np.array_equal(bits16(lin.w_dense), od)
    assert np.array_equal(canonical_meta(ctx, lin.meta, O, I, B.BF16), om)
    ogv, ogm, _, _ = orc.mvue(dY, cfg["seed"], layer, 3)
    assert np.array_equal(bits16(lin.gvals), ogv)
    assert np.array_equal(canonical_meta(ctx, lin.gmeta, O, T, B.BF16), ogm)
    for got, ref in ((lin.Y, orc.linear_fwd(X, orc.BF16, ov, om, orc.BF16)),
                     (lin.dW, orc.linear_bwd_weight(ogv, ogm, orc.BF16, X, orc.BF16)),
                     (lin.dX, orc.linear_bwd_input(dY, orc.BF16, od, orc.BF16))):
        g = got.float().cpu().numpy()
        assert rel_fro(g, ref) <= BF16_GEMM_TOL
        assert (np.abs(g - ref) <= 2.0 ** -7 * np.abs(ref) + 1e-4 * np.abs(ref).max()).all()


def _sampled_products(lin, X_dec, dY_dec, w_dec, vals, meta, gvals, gmeta, wdt, gdt, inv, tol, rng):
    """Compare N_SAMPLE rows of Y, dW and dX with fp64 dot products of the decoded operands."""
    T, O, I = X_dec.shape[0], w_dec.shape[0], w_dec.shape[1]
    ts = np.sort(rng.choice(T, N_SAMPLE, replace=False))
    os_ = np.sort(rng.choice(O, N_SAMPLE, replace=False))
    idx_t = torch.from_numpy(ts).to(DEV)
    idx_o = torch.from_numpy(os_).to(DEV)
    Y_ref = (X_dec[ts] @ w_dec.T) * inv["xw"]
    dX_ref = (dY_dec[ts] @ w_dec) * inv["gw"]
    G_rows = orc.decompress(np.ascontiguousarray(gvals[os_]), np.ascontiguousarray(gmeta[os_]), gdt).astype(np.float64)
    dW_ref = (G_rows @ X_dec) * inv["gx"]
    assert rel_fro(lin.Y[idx_t].float().cpu().numpy(), Y_ref) <= tol
    assert rel_fro(lin.dX[idx_t].float().cpu().numpy(), dX_ref) <= tol
    assert rel_fro(lin.dW[idx_o].float().cpu().numpy(), dW_ref) <= tol
    # the dense copy used by grad_X is the decompressed operand of the forward
    assert np.array_equal(orc.decompress(np.ascontiguousarray(vals[os_]), np.ascontiguousarray(meta[os_]), wdt).astype(np.float64),
                          w_dec[os_])


def _bf16_layer_sampled(ctx, cfg_id, layer, rng_seed):
    """One bf16 layer at full size: beta, projection, metadata and MVUE in full and bit for bit; the three
    products on N_SAMPLE rows each against fp64 dot products."""
    from paper_2409_09099_b200 import binding as B
    cfg = synth.CONFIGS[cfg_id]
    W, X, dY = synth.layer_tensors(cfg_id, layer)
    O, I = W.shape
    T = X.shape[0]
    lin = _run_layer(ctx, W, X, dY, layer, cfg["seed"], 0, False)
    beta_ref = orc.beta(W)[0]
    assert abs(lin.beta.item() - beta_ref) <= 1e-6 * beta_ref
    ov, om, od = orc.project_compress(W, np.float32(lin.beta.item()))
    assert np.array_equal(bits16(lin.vals), ov) and np.array_equal(bits16(lin.w_dense), od)
    assert np.array_equal(canonical_meta(ctx, lin.meta, O, I, B.BF16), om)
    ogv, ogm, _, _ = orc.mvue(dY, cfg["seed"], layer, 0)
    assert np.array_equal(bits16(lin.gvals), ogv)
    assert np.array_equal(canonical_meta(ctx, lin.gmeta, O, T, B.BF16), ogm)
    _sampled_products(lin, orc.decode(X, orc.BF16), orc.decode(dY, orc.BF16), orc.decode(od, orc.BF16), ov, om, ogv, ogm,
                      orc.BF16, orc.BF16, dict(xw=1.0, gw=1.0, gx=1.0), BF16_GEMM_TOL, np.random.default_rng(rng_seed))


# GPT-2-large block linears, 16384 tokens: qkv [3840, 1280], proj [1280, 1280], fc1 [5120, 1280], fc2 [1280, 5120]
@pytest.mark.parametrize("layer", [0, 1, 2, 3])
def test_config3_every_layer_sampled(ctx, layer):
    _bf16_layer_sampled(ctx, 3, layer, 30 + layer)


# the attention linears of a GPT-2-124M block, 8192 tokens: qkv [2304, 768], proj [768, 768] (its MLP layers have
# the shapes of config 2, which is compared in full above)
@pytest.mark.parametrize("layer", [0, 1])
def test_config4_attention_linears_sampled(ctx, layer):
    _bf16_layer_sampled(ctx, 4, layer, 40 + layer)


# FP8 whole-process, 7B-shaped FFN, 16384 tokens: up / gate [11008, 4096] and down [4096, 11008] (K = 11008: an odd
# number of pipeline stages and its own tile-width / split plan)
@pytest.mark.parametrize("layer", [0, 1, 2])
def test_config5_fp8_every_layer_sampled(ctx, layer):
    from paper_2409_09099_b200 import binding as B
    cfg = synth.CONFIGS[5]
    W, X, dY = synth.layer_tensors(5, layer)
    O, I = W.shape
    T = X.shape[0]
    lin = _run_layer(ctx, W, X, dY, layer, cfg["seed"], 0, True)
    beta32 = np.float32(lin.beta.item())
    assert abs(float(beta32) - orc.beta(W)[0]) <= 1e-6 * float(beta32)
    _, _, wt16 = orc.project_compress(W, beta32)
    sw, sx, sg = (orc.fp8_scale(orc.amax(wt16), orc.E4M3), orc.fp8_scale(orc.amax(X), orc.E4M3),
                  orc.fp8_scale(orc.amax(dY), orc.E5M2))
    assert lin.amax.cpu().numpy().tolist() == [orc.amax(X), orc.amax(wt16), orc.amax(dY)]
    ov, om, od = orc.project_compress(W, beta32, odt=orc.E4M3, wscale=sw)
    assert np.array_equal(bits8(lin.vals), ov) and np.array_equal(bits8(lin.w_dense), od)
    assert np.array_equal(canonical_meta(ctx, lin.meta, O, I, B.E4M3), om)
    Xq = orc.quantize(X, sx, orc.E4M3)
    assert np.array_equal(bits8(lin.Xq), Xq)
    ogv, ogm, odq, _ = orc.mvue(dY, cfg["seed"], layer, 0, odt=orc.E5M2, gscale=sg, want_dense_q=True)
    assert np.array_equal(bits8(lin.gvals), ogv) and np.array_equal(bits8(lin.dYq), odq)
    assert np.array_equal(canonical_meta(ctx, lin.gmeta, O, T, B.E5M2), ogm)
    inv = dict(xw=1.0 / (float(sx) * float(sw)), gw=1.0 / (float(sg) * float(sw)), gx=1.0 / (float(sg) * float(sx)))
    _sampled_products(lin, orc.decode(Xq, orc.E4M3), orc.decode(odq, orc.E5M2), orc.decode(od, orc.E4M3), ov, om, ogv, ogm,
                      orc.E4M3, orc.E5M2, inv, FP8_GEMM_TOL, np.random.default_rng(50 + layer))
