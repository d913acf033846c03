"""sste_beta_init_static: the beta reduction for callers that cannot allocate device memory.

Such callers (a runtime that owns the whole memory pool, a plug-in that only sees its inputs and outputs,
a job on a full device) have no workspace to give the library and so no context; the entry point keeps its
scratch in a fixed array inside libsste.so instead.  The test calls it through the C ABI twice in a row, on
tensors of different sizes so that the second call meets the first call's leftovers in the shared array, and
checks both results against the context-based sste_beta_init and against the CPU oracle's fp64 beta, within the
beta tolerance of the other GPU tests.
This file sorts last on purpose: a run that stops at the first failure has then run every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import sste_oracle as orc
from paper_2409_09099_b200 import synth

pytestmark = pytest.mark.gpu

BETA_TOL = 1e-6     # relative; the two calls sum the same fp64 terms in different orders
DEV = "cuda:0"


def _dbf16(a):
    return torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).to(DEV).view(torch.bfloat16)


def test_static_scratch_beta_matches_context_beta_twice():
    from paper_2409_09099_b200 import binding as B
    ctx = B.Context(0)
    # the very first call makes the driver load the kernel and the scratch array with it (lazy module
    # loading); from then on the free device memory must not move
    warm = torch.zeros(1, dtype=torch.float32, device=DEV)
    B.beta_init_static(torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV), warm)
    torch.cuda.synchronize()
    # first a large tensor (1032 tiles), then a small one (6 tiles): stale partials beyond the second
    # call's tiles and a used ticket counter must not leak into its result
    for seed, (O, I) in ((1, (3072, 5504)), (2, (256, 384))):
        W_host = synth.gaussian_bf16(seed, (O, I), 0.02)
        W = _dbf16(W_host)
        want = torch.zeros(1, dtype=torch.float32, device=DEV)
        got = torch.full((1,), -1.0, dtype=torch.float32, device=DEV)
        ctx.beta_init(W, want)
        torch.cuda.synchronize()
        free_before, held_before = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated()
        B.beta_init_static(W, got)
        torch.cuda.synchronize()
        # free memory may rise if another process on a shared GPU releases some; it must not fall
        assert torch.cuda.mem_get_info()[0] >= free_before, "the call must not allocate device memory"
        assert torch.cuda.memory_allocated() == held_before
        assert abs(got.item() - want.item()) <= BETA_TOL * abs(want.item()), (got.item(), want.item())
        ref = orc.beta(W_host)[0]                       # Eq. 5 in fp64 on the CPU
        assert abs(got.item() - ref) <= BETA_TOL * abs(ref), (got.item(), ref)
        # reproducible: the partials are combined in tile order
        again = torch.zeros(1, dtype=torch.float32, device=DEV)
        B.beta_init_static(W, again)
        assert again.item() == got.item()
    # already 2:4-sparse weights project onto themselves: beta = 1 exactly; all-equal groups: S_soft = 0 -> 1
    Wf = synth.bf16_bits_to_f32(synth.gaussian_bf16(3, (128, 256), 0.02)).reshape(128, 64, 4)
    Wf[:, :, [0, 2]] = 0
    out = torch.zeros(1, dtype=torch.float32, device=DEV)
    B.beta_init_static(_dbf16(synth.to_bf16_bits(Wf.reshape(128, 256))), out)
    assert out.item() == 1.0
    B.beta_init_static(_dbf16(synth.to_bf16_bits(np.full((128, 128), 0.5, np.float32))), out)
    assert out.item() == 1.0
    assert ctx.poll_device_status() == 0
    ctx.close()


def test_static_scratch_rejects_what_does_not_fit():
    from paper_2409_09099_b200 import binding as B
    lib = B.load()
    W = torch.zeros((128, 128), dtype=torch.bfloat16, device=DEV)
    out = torch.zeros(1, dtype=torch.float32, device=DEV)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    args = (ctypes.c_void_p(W.data_ptr()),)
    # 8192 tiles fit; one tile row more does not (refused before anything is launched, W is not touched)
    assert lib.sste_beta_init_static(0, *args, 128 * 8193, 128, B.BF16, ctypes.c_void_p(out.data_ptr()), stream) == B.ERR_WORKSPACE
    assert lib.sste_beta_init_static(0, *args, 16384, 16384, B.BF16, ctypes.c_void_p(out.data_ptr()), stream) == B.ERR_WORKSPACE
    assert lib.sste_beta_init_static(0, *args, 192, 128, B.BF16, ctypes.c_void_p(out.data_ptr()), stream) == B.ERR_SHAPE
    assert lib.sste_beta_init_static(0, None, 128, 128, B.BF16, ctypes.c_void_p(out.data_ptr()), stream) == B.ERR_INVALID_ARG
    assert lib.sste_beta_init_static(0, *args, 128, 128, B.E4M3, ctypes.c_void_p(out.data_ptr()), stream) == B.ERR_DTYPE
    assert lib.sste_beta_init_static(0, *args, 128, 128, B.BF16, ctypes.c_void_p(out.data_ptr()), stream) == B.OK
    torch.cuda.synchronize()
    assert out.item() == 1.0        # all-zero weights: S_soft = 0, beta defined as 1
