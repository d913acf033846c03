"""Config 4: a 12-layer GPT-2-124M-shaped decoder with all 48 linear layers routed through libsste, 10 training
steps on a fixed synthetic batch of uniform token ids.

Parity is checked per call: at steps 0 and 9 every S-STE linear's calls are replayed through the CPU oracle on the
tensors the model actually fed them -- beta (Eq. 5; computed at step 0 only and frozen, Sec. 4.2), projection,
metadata and MVUE (with the step counter of that iteration) bit for bit, the three products on sampled rows
against fp64 dot products.  The run also checks what only a multi-step, multi-layer run exercises: one context
shared by 48 layers, the straight-through update of the dense weights (Eq. 3) changing the projection between
steps while beta stays fixed, a finite loss that starts near ln(50257) and falls on the memorised batch.
"""
import math

import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from tests.gpu_util import DEV, bits16, canonical_meta, rel_fro

pytestmark = pytest.mark.gpu

N_ROWS = 48          # sampled output rows per product


def test_config4_ten_training_steps_with_per_call_replay():
    from paper_2409_09099_b200 import binding as B
    from paper_2409_09099_b200.model import SsteGpt2, synthetic_batch
    ctx = B.Context(0)
    model = SsteGpt2(ctx)
    tokens, targets = synthetic_batch(model, 4)
    assert len(model.linears) == 48
    beta0, seen = {}, {0: set(), 9: set()}
    rng = np.random.default_rng(44)

    def replay(index, step, lin, x, dy):
        assert step == model.step_index
        if step not in seen:
            return
        torch.cuda.synchronize()
        seen[step].add(index)
        O, I, T = lin.O, lin.I, lin.T
        W, X, dY = bits16(lin.W), bits16(x), bits16(dy)
        beta32 = np.float32(lin.beta.item())
        if step == 0:
            ref = orc.beta(W)[0]
            assert abs(float(beta32) - ref) <= 1e-6 * ref
            beta0[index] = beta32
        else:
            assert beta32 == beta0[index]                       # frozen after the first iteration
            assert abs(orc.beta(W)[0] - float(beta32)) > 0      # ... although the weights have moved
        ov, om, od = orc.project_compress(W, beta32)
        assert np.array_equal(bits16(lin.vals), ov) and np.array_equal(bits16(lin.w_dense), od)
        assert np.array_equal(canonical_meta(ctx, lin.meta, O, I, B.BF16), om)
        ogv, ogm, _, _ = orc.mvue(dY, model.seed, index, step)
        assert np.array_equal(bits16(lin.gvals), ogv)
        assert np.array_equal(canonical_meta(ctx, lin.gmeta, O, T, B.BF16), ogm)
        ts = np.sort(rng.choice(T, N_ROWS, replace=False))
        os_ = np.sort(rng.choice(O, N_ROWS, replace=False))
        it, io = torch.from_numpy(ts).to(DEV), torch.from_numpy(os_).to(DEV)
        Xd, Gd, Wd = orc.decode(X, orc.BF16), orc.decode(dY, orc.BF16), orc.decode(od, orc.BF16)
        assert rel_fro(lin.Y[it].float().cpu().numpy(), Xd[ts] @ Wd.T) <= 1e-2
        assert rel_fro(lin.dX[it].float().cpu().numpy(), Gd[ts] @ Wd) <= 1e-2
        G_rows = orc.decompress(np.ascontiguousarray(ogv[os_]), np.ascontiguousarray(ogm[os_]), orc.BF16).astype(np.float64)
        assert rel_fro(lin.dW[io].float().cpu().numpy(), G_rows @ Xd) <= 1e-2

    model.on_call = replay
    losses, inside, total = [], 0.0, 0.0
    w_before = model.linears[0].w.detach().clone()
    for step in range(10):
        timed = step in (3, 4, 5)                               # steps without replay: time inside libsste
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        loss, t_in = model.train_step(tokens, targets, time_libsste=timed)
        e1.record()
        torch.cuda.synchronize()
        losses.append(float(loss))
        if timed:
            inside += t_in
            total += e0.elapsed_time(e1) * 1e-3
    assert all(math.isfinite(v) for v in losses)
    assert abs(losses[0] - math.log(50257.0)) < 0.6             # uniform random tokens, random init
    assert losses[-1] < losses[0]                               # the fixed batch is being memorised
    assert seen[0] == set(range(48)) and seen[9] == set(range(48))
    assert all(s.beta_launches == 1 for s in model.linears)     # beta computed in the first iteration only
    assert not torch.equal(model.linears[0].w.detach(), w_before)   # grad_W reached the dense weight (Eq. 3)
    frac = inside / total
    assert 0.0 < frac < 1.0
    print(f"config 4: losses {losses[0]:.3f} -> {losses[-1]:.3f}; {100 * frac:.1f} % of the step inside libsste "
          f"({1e3 * total / 3:.1f} ms per step)")
    assert ctx.poll_device_status() == 0
    ctx.close()
