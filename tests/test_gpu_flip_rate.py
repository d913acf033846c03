"""GPU parity of the flip count (Sec. 3.1, "Flip rate") against the oracle's definition on the dense weights."""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, dbf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    from paper_2409_09099_b200 import binding
    c = binding.Context(0)
    yield c
    assert c.poll_device_status() == 0
    c.close()


def _perturbed(W, sigma, seed):
    f = orc.bf16_to_f32(W)
    rng = np.random.default_rng(seed)
    return orc.f32_to_bf16((f + sigma * rng.standard_normal(f.shape)).astype(np.float32))


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("O,I,sigma", [(128, 128, 1e-3), (384, 640, 5e-3), (3072, 768, 2e-4), (256, 1024, 0.0)])
def test_flip_count_matches_the_definition(ctx, O, I, sigma, fp8):
    from paper_2409_09099_b200 import binding as B
    W0 = synth.gaussian_bf16(O + I, (O, I), 0.02)
    W0[: O // 8].reshape(-1, 4)[:, :] = W0[: O // 8].reshape(-1, 4)[:, :1]        # all-equal groups: tie rule decides
    W1 = _perturbed(W0, sigma, 3) if sigma > 0 else W0.copy()
    dt = B.E4M3 if fp8 else B.BF16
    beta = torch.full((1,), 1.3, dtype=torch.float32, device=DEV)
    unit = torch.full((1,), 448.0, dtype=torch.float32, device=DEV)       # amax 448: E4M3 scale 1
    metas = []
    for W in (W0, W1):
        vals, meta = ctx.alloc_compressed(O, I, dt)
        ctx.project_compress(dbf16(W), beta, vals, meta, None, w_amax_dev=unit if fp8 else None)
        metas.append(meta)
    count = torch.full((1,), -1, dtype=torch.int64, device=DEV)
    for _ in range(2):                                        # the call zeroes its own counter
        ctx.flip_count(metas[0], metas[1], O, I, count)
    want = orc.flip_count(W0, W1)
    assert int(count.item()) == want
    assert (want == 0) == (sigma == 0.0)


def test_layer_tracks_flip_rate(ctx):
    from paper_2409_09099_b200.layer import SsteLinear
    O, I, T = 256, 512, 128
    W0 = synth.gaussian_bf16(21, (O, I), 0.02)
    W1 = _perturbed(W0, 2e-3, 4)
    Wd = dbf16(W0)
    lin = SsteLinear(ctx, Wd, T, track_flips=True)
    lin.init_beta()
    lin.prune()
    assert lin.flip_rate() == 0.0
    Wd.copy_(dbf16(W1))                                       # the optimiser's update of the dense weight
    lin.prune()
    assert lin.flip_rate() == orc.flip_rate(W0, W1)
    lin.prune()                                               # nothing changed since
    assert lin.flip_rate() == 0.0


def test_argument_checks(ctx):
    from paper_2409_09099_b200 import binding as B
    m = torch.zeros(2048, dtype=torch.uint8, device=DEV)
    c = torch.zeros(1, dtype=torch.int64, device=DEV)
    with pytest.raises(B.SsteError) as e:
        ctx.flip_count(m, m, 100, 128, c)
    assert e.value.code == B.ERR_SHAPE
