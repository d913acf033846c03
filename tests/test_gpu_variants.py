"""GPU parity of the ablation variants of the pruning step (interpolated threshold, hard threshold, L1 beta,
SR-STE decay) against the oracle: bit-exact outputs, beta to 1e-6."""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, bits8, canonical_meta, dbf16, rel_fro

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def _weights(O, I, seed):
    W = synth.gaussian_bf16(seed, (O, I), 0.02)
    g = W[: O // 4].reshape(-1, 4)
    g[0::4, 1] = g[0::4, 2]                      # ties between the second and third magnitude
    g[1::4, :] = g[1::4, :1]                     # all-equal groups
    g[2::4, 2:] = 0                              # already 2:4
    g[3::4, 0] = 0x8000                          # -0
    return W


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("hard,gamma", [(False, 0.0), (False, 0.25), (False, 0.5), (False, 1.0), (True, 0.0)])
@pytest.mark.parametrize("O,I", [(128, 128), (384, 640)])
def test_projection_variants(ctx, O, I, hard, gamma, fp8):
    from paper_2409_09099_b200 import binding as B
    W = _weights(O, I, O + I)
    beta32 = np.float32(1.0 if hard else 1.4837)
    w_amax = np.float32(4.90625)                       # the kernel forms the scale 448 / amax itself
    ws = orc.fp8_scale(w_amax, orc.E4M3)
    dt = B.E4M3 if fp8 else B.BF16
    odt = orc.E4M3 if fp8 else orc.BF16
    beta = torch.full((1,), float(beta32), dtype=torch.float32, device=DEV)
    wsd = torch.full((1,), float(w_amax), dtype=torch.float32, device=DEV)
    vals, meta = ctx.alloc_compressed(O, I, dt)
    dense = torch.empty((O, I), dtype=B._TORCH_DT[dt], device=DEV)
    ctx.project_compress_variant(dbf16(W), beta, vals, meta, dense, w_amax_dev=wsd if fp8 else None, hard=hard,
                                 gamma=gamma)
    ov, om, od = orc.project_compress_variant(W, beta32, gamma=gamma, hard=hard, odt=odt, wscale=ws)
    bits = bits8 if fp8 else bits16
    assert np.array_equal(bits(vals), ov)
    assert np.array_equal(bits(dense), od)
    assert np.array_equal(canonical_meta(ctx, meta, O, I, dt), om)


def test_gamma_zero_runs_the_default_kernel(ctx):
    from paper_2409_09099_b200 import binding as B
    O, I = 256, 256
    W = dbf16(_weights(O, I, 5))
    beta = torch.full((1,), 1.25, dtype=torch.float32, device=DEV)
    a, am = ctx.alloc_compressed(O, I)
    b, bm = ctx.alloc_compressed(O, I)
    ctx.project_compress(W, beta, a, am)
    ctx.project_compress_variant(W, beta, b, bm, gamma=0.0)
    assert torch.equal(a.view(torch.int16), b.view(torch.int16)) and torch.equal(am, bm)
    with pytest.raises(B.SsteError) as e:
        ctx.project_compress_variant(W, beta, b, bm, gamma=1.5)
    assert e.value.code == B.ERR_INVALID_ARG


def test_beta_l1(ctx):
    W = _weights(384, 640, 17)
    beta = torch.zeros(1, dtype=torch.float32, device=DEV)
    ctx.beta_init_l1(dbf16(W), beta)
    ref = orc.beta_l1(W)
    assert abs(beta.item() - ref) <= 1e-6 * ref
    first = beta.item()
    ctx.beta_init_l1(dbf16(W), beta)             # reproducible
    assert beta.item() == first
    ctx.beta_init(dbf16(W), beta)                # and distinct from the MSE-optimal scale
    assert beta.item() < first


@pytest.mark.parametrize("fp8", [False, True])
def test_srste_decay(ctx, fp8):
    from paper_2409_09099_b200 import binding as B
    O, I, lam = 256, 384, 2e-4
    W = _weights(O, I, 23)
    dW = synth.gaussian_bf16(24, (O, I), 1e-3)
    dt = B.E4M3 if fp8 else B.BF16
    one = torch.ones(1, dtype=torch.float32, device=DEV)
    vals, meta = ctx.alloc_compressed(O, I, dt)
    unit = torch.full((1,), 448.0, dtype=torch.float32, device=DEV)       # amax 448: E4M3 scale 1
    ctx.project_compress(dbf16(W), one, vals, meta, None, w_amax_dev=unit if fp8 else None)
    g = dbf16(dW)
    ctx.srste_decay(dbf16(W), meta, dt, lam, g)
    assert np.array_equal(bits16(g), orc.srste_decay(dW, W, lam))


def test_grad_input_with_mvue_on_the_weight(ctx):
    """The rejected ablation of Sec. 5.1 (MVUE on S(W) for grad_X), composed of existing calls: operand bits equal
    the oracle's MVUE of w~ along O, the product matches fp64, and the estimator is unbiased over steps."""
    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.layer import SsteLinear
    O, I, T = 256, 384, 512
    W = synth.gaussian_bf16(31, (O, I), 0.02)
    X = synth.gaussian_bf16(32, (T, I), 1.0)
    dY = synth.gaussian_bf16(33, (T, O), 1e-2)
    lin = SsteLinear(ctx, dbf16(W), T, tensor_id=2, seed=5)
    lin.init_beta(); lin.prune(); lin.forward(dbf16(X))
    lin.grad_input_mvue_weight(dbf16(dY), step=4)
    torch.cuda.synchronize()
    _, _, wt = orc.project_compress(W, np.float32(lin.beta.item()))
    ogv, ogm, _, _ = orc.mvue(wt, 5, 2 + (1 << 16), 4)                   # w~ [O, I] sparsified along O -> [I, O]
    assert np.array_equal(bits16(lin.wt_vals), ogv)
    assert np.array_equal(canonical_meta(ctx, lin.wt_meta, I, O, B.BF16), ogm)
    ref = orc.linear_fwd(dY, orc.BF16, ogv, ogm, orc.BF16)               # dX[T, I] = dY MVUE(w~^T)^T
    assert rel_fro(lin.dX.float().cpu().numpy(), ref) <= 1e-2
    # unbiased: the mean over steps approaches the dense grad_X (statistical bound: 6 sigma of the sample mean)
    exact = orc.linear_bwd_input(dY, orc.BF16, wt, orc.BF16)
    acc = np.zeros_like(exact)
    n = 64
    for s in range(n):
        lin.grad_input_mvue_weight(dbf16(dY), step=100 + s)
        acc += lin.dX.float().cpu().numpy()
    err = np.linalg.norm(acc / n - exact) / np.linalg.norm(exact)
    one = np.linalg.norm(lin.dX.float().cpu().numpy() - exact) / np.linalg.norm(exact)
    assert err < 6.0 * one / np.sqrt(n) + 5e-3
