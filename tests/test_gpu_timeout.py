"""A bounded device-side wait that runs out: the kernel gives up, reports, and the context stays usable.

Every wait inside the product kernels carries a wall-clock limit.  The test hook sste_debug_inject_stall makes the
operand producer of a one-tile dense grad_X product leave its last pipeline stage unloaded (a barrier that nothing
completes) with the limit shortened to a millisecond.  The call must return, the status word must read
SSTE_ERR_TIMEOUT, and the next ordinary call on the same context must be correct bit for bit.  Nothing here
faults, traps or spins: the kernel's own bounded waits end it.
"""
import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth
from tests.gpu_util import DEV, bits16, dbf16, rel_fro

pytestmark = pytest.mark.gpu


def test_expired_wait_is_reported_and_the_context_survives():
    from paper_2409_09099_b200 import binding as B
    ctx = B.Context(0)
    T, O, I = 128, 256, 128                      # one 256 x 256 output tile, four K stages
    dY = synth.gaussian_bf16(1, (T, O), 1e-2)
    Wd = synth.gaussian_bf16(2, (O, I), 0.02)
    dYd, Wdd = dbf16(dY), dbf16(Wd)
    dX = torch.zeros((T, I), dtype=torch.bfloat16, device=DEV)
    ref = orc.linear_bwd_input(dY, orc.BF16, Wd, orc.BF16)
    ctx.linear_bwd_input(dYd, Wdd, dX)           # healthy call first
    torch.cuda.synchronize()
    good = bits16(dX).copy()
    assert rel_fro(dX.float().cpu().numpy(), ref) <= 1e-2
    assert ctx.poll_device_status() == B.OK

    ctx.debug_inject_stall(True)
    try:
        # while armed, any other product refuses before launching anything
        vals, meta = ctx.alloc_compressed(O, I)
        with pytest.raises(B.SsteError):
            ctx.linear_bwd_input(dYd, None, dX, vals=vals, meta=meta)
        dX.zero_()
        ctx.linear_bwd_input(dYd, Wdd, dX)       # the wait for the unloaded stage runs out after ~1 ms
        torch.cuda.synchronize()                 # the kernel has returned
    finally:
        ctx.debug_inject_stall(False)
    assert ctx.poll_device_status() == B.ERR_TIMEOUT
    assert ctx.poll_device_status() == B.OK      # reading the word clears it

    dX.zero_()
    ctx.linear_bwd_input(dYd, Wdd, dX)           # the same context, an ordinary call: bit-identical to before
    torch.cuda.synchronize()
    assert np.array_equal(bits16(dX), good)
    assert ctx.poll_device_status() == B.OK
    ctx.close()
