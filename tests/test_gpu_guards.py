"""Guard bands around every output: no kernel of the path writes outside the tensors it was given.

The memory checker of the CUDA toolkit is not available on the GPU pool, so the check is done by hand: each output
lives inside a larger allocation with 4 KB of a known byte pattern before and after it, and the pattern must be
intact after the calls.  Shapes include partial tiles (384, 640, 1152) and tile widths that do not divide the
problem (224), where out-of-range rows and columns are handled by the clipping of the bulk stores.
"""
import numpy as np
import pytest
import torch

from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, dbf16

pytestmark = pytest.mark.gpu

GUARD = 4096
PATTERN = 0xA5


class Guarded:
    def __init__(self):
        self.bufs = []

    def alloc(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        pad = (-n) % 128
        raw = torch.full((GUARD + n + pad + GUARD,), PATTERN, dtype=torch.uint8, device=DEV)
        self.bufs.append((raw, n))
        return raw[GUARD:GUARD + n].view(dtype).view(shape)

    def check(self):
        for raw, n in self.bufs:
            assert bool((raw[:GUARD] == PATTERN).all()), "write before an output"
            assert bool((raw[GUARD + n:] == PATTERN).all()), "write past an output"


@pytest.mark.parametrize("fp8", [False, True])
@pytest.mark.parametrize("O,I,T,bn", [(128, 128, 128, 0), (384, 640, 1152, 0), (384, 640, 1152, 224), (640, 384, 384, 128),
                                      (256, 1152, 640, 192)])
def test_no_call_writes_outside_its_outputs(O, I, T, bn, fp8):
    from paper_2409_09099_b200 import binding as B
    ctx = B.Context(0)
    g = Guarded()
    f32 = dict(dtype=torch.float32, device=DEV)
    W, X, dY = (dbf16(synth.gaussian_bf16(s, shp, sig)) for s, shp, sig in
                ((1, (O, I), 0.02), (2, (T, I), 1.0), (3, (T, O), 1e-2)))
    wdt, gdt = (torch.float8_e4m3fn, torch.float8_e5m2) if fp8 else (torch.bfloat16, torch.bfloat16)
    beta, amax = g.alloc((1,), torch.float32), g.alloc((3,), torch.float32)
    vals, meta = g.alloc((O, I // 2), wdt), g.alloc((O * I // 8,), torch.uint8)
    dense, dec = g.alloc((O, I), wdt), g.alloc((O, I), wdt)
    gvals, gmeta = g.alloc((O, T // 2), gdt), g.alloc((O * T // 8,), torch.uint8)
    Xq = g.alloc((T, I), torch.float8_e4m3fn) if fp8 else X
    dYq = g.alloc((T, O), torch.float8_e5m2) if fp8 else None
    Y, dX, dX2, dW = (g.alloc(s, torch.bfloat16) for s in ((T, O), (T, I), (T, I), (O, I)))
    out_amax = g.alloc((2,), torch.float32)
    canon = g.alloc((O, I // 16), torch.int16)
    ax, aw, ag = (amax[0:1], amax[1:2], amax[2:3]) if fp8 else (None, None, None)
    ctx.debug_force_tile_width(bn)
    try:
        ctx.beta_init(W, beta)
        if fp8:
            ctx.project_amax(W, beta, aw)
            ctx.amax(X, ax)
            ctx.amax(dY, ag)
            ctx.quantize_fp8(X, ax, Xq)
        ctx.project_compress(W, beta, vals, meta, dense, w_amax_dev=aw)
        ctx.decompress(vals, meta, dec)
        ctx.meta_to_canonical(meta, O, I, B.E4M3 if fp8 else B.BF16, canon)
        ctx.linear_fwd(Xq, vals, meta, Y, x_amax_dev=ax, w_amax_dev=aw, y_amax_out_dev=out_amax[0:1])
        ctx.mvue_sparsify(dY, 3, 1, 2, gvals, gmeta, dense_q_out=dYq, g_amax_dev=ag)
        ctx.linear_bwd_weight(gvals, gmeta, Xq, dW, g_amax_dev=ag, x_amax_dev=ax)
        ctx.linear_bwd_input(dYq if fp8 else dY, dense, dX, g_amax_dev=ag, w_amax_dev=aw, dx_amax_out_dev=out_amax[1:2])
        ctx.linear_bwd_input(dYq if fp8 else dY, None, dX2, g_amax_dev=ag, w_amax_dev=aw, vals=vals, meta=meta)
        torch.cuda.synchronize()
    finally:
        ctx.debug_force_tile_width(0)
    g.check()
    assert torch.equal(dX.view(torch.int16), dX2.view(torch.int16))
    assert ctx.poll_device_status() == 0
    ctx.close()
