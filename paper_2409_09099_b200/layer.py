"""One S-STE linear layer as a user of the library sees it: buffers + the call sequence.

This is bookkeeping only (which buffer goes to which C-ABI call, in the order the
paper's training iteration prescribes); every computation runs in libsste.
Straight-through estimator (Eq. 3): ``dW`` is the gradient with respect to the
sparse weight and is meant to be applied to the dense weight unchanged.
"""
from __future__ import annotations

import torch

from . import binding as B


class SsteLinear:
    """W[O, I] dense master weight (bf16); forward Y = X S(W)^T, backward (dX, dW).

    ``fp8=True`` selects the whole-process FP8 variant (Sec. 5.2): E4M3 forward
    operands, E5M2 output gradient, per-tensor scale = fp8_max / amax; the state of a
    quantised tensor is its amax (one device float), from which every consumer forms the
    scale itself.  ``dense_copy=True`` (the default, the faster route on B200) also keeps w~ as a
    dense [O, I] tensor and feeds grad_X from it; with ``dense_copy=False`` no dense w~ exists and
    grad_X expands the compressed operand inside the product (same bits, less memory, slower).
    ``track_flips=True`` keeps the previous iteration's metadata and counts the mask entries
    that changed at every prune (flip rate, Sec. 3.1).
    """

    def __init__(self, ctx: B.Context, W: torch.Tensor, T: int, tensor_id: int = 0, seed: int = 0,
                 fp8: bool = False, out_dtype: torch.dtype = torch.bfloat16, track_flips: bool = False,
                 dense_copy: bool = True, counter_cols: int = 0):
        assert W.dtype == torch.bfloat16 and W.is_cuda
        self.ctx, self.W, self.T, self.tensor_id, self.seed, self.fp8 = ctx, W, T, tensor_id, seed, fp8
        self.O, self.I = W.shape
        self.counter_cols = counter_cols
        O, I, dev = self.O, self.I, W.device
        f32 = dict(dtype=torch.float32, device=dev)
        self.beta = torch.zeros(1, **f32)
        self.beta_ready = False
        wdt = B.E4M3 if fp8 else B.BF16
        gdt = B.E5M2 if fp8 else B.BF16
        self.vals, self.meta = ctx.alloc_compressed(O, I, wdt)
        self.w_dense = torch.empty((O, I), dtype=B._TORCH_DT[wdt], device=dev) if dense_copy else None
        self.gvals, self.gmeta = ctx.alloc_compressed(O, T, gdt)
        self.Y = torch.empty((T, O), dtype=out_dtype, device=dev)
        self.dX = torch.empty((T, I), dtype=out_dtype, device=dev)
        self.dW = torch.empty((O, I), dtype=out_dtype, device=dev)
        self.launches = 0
        self.mark = None       # optional callback(label), called before every C-ABI call (a benchmark records events)
        self.track_flips = track_flips
        if track_flips:
            self.meta_prev = torch.empty_like(self.meta)
            self.flips = torch.zeros(1, dtype=torch.int64, device=dev)   # mask entries changed by the last prune
            self._have_prev = False
        self.amax = torch.zeros(3, **f32) if fp8 else None     # max|X|, max|w~| (bf16 projection), max|dY|
        if fp8:
            self.Xq = torch.empty((T, I), dtype=torch.float8_e4m3fn, device=dev)
            self.dYq = torch.empty((T, O), dtype=torch.float8_e5m2, device=dev)

    def _amax(self, k):
        return self.amax[k:k + 1] if self.fp8 else None

    def _m(self, label):
        if self.mark is not None:
            self.mark(label)

    # (0) first iteration only: beta is computed once and then frozen (Sec. 4.2)
    def init_beta(self):
        self.ctx.beta_init(self.W, self.beta)
        self.beta_ready = True
        self.launches += 1

    # (1) prune: w~ = beta * S_soft(W), compressed for the sparse products (and for grad_X)
    def prune(self):
        assert self.beta_ready, "call init_beta() in the first iteration"
        c = self.ctx
        if self.track_flips:
            self.meta, self.meta_prev = self.meta_prev, self.meta     # last iteration's image becomes "previous"
        if self.fp8:
            # the scale of w~ needs amax(w~) first: one read-only pass over W, then the cast to E4M3
            self._m("project_amax")
            c.project_amax(self.W, self.beta, self.amax[1:2])
            self.launches += 1
        self._m("project_compress")
        c.project_compress(self.W, self.beta, self.vals, self.meta, self.w_dense, w_amax_dev=self._amax(1))
        self.launches += 1
        if self.track_flips:
            if self._have_prev:
                self._m("flip_count")
                c.flip_count(self.meta_prev, self.meta, self.O, self.I, self.flips)
                self.launches += 1
            self._have_prev = True

    def flip_rate(self) -> float:
        """r_k of the last prune (synchronises); 0 before the second prune."""
        return float(self.flips.item()) / (self.O * self.I)

    # (2a) forward with the sparse weight
    def forward(self, X, y_amax_out=None):
        c = self.ctx
        if not self.fp8:
            self.X = X
            self._m("linear_fwd")
            c.linear_fwd(X, self.vals, self.meta, self.Y, y_amax_out_dev=y_amax_out)
            self.launches += 1
            return self.Y
        self._m("amax_x")
        c.amax(X, self.amax[0:1])
        self._m("quantize_x")
        c.quantize_fp8(X, self.amax[0:1], self.Xq)
        self._m("linear_fwd")
        c.linear_fwd(self.Xq, self.vals, self.meta, self.Y, x_amax_dev=self.amax[0:1], w_amax_dev=self.amax[1:2],
                     y_amax_out_dev=y_amax_out)
        self.launches += 3
        return self.Y

    # (2b) backward: MVUE on the output gradient for grad_W, dense product for grad_X
    def backward(self, dY, step: int = 0, token_offset: int = 0):
        self.sparsify_grad(dY, step, token_offset)
        self.grad_weight()
        self.grad_input(dY)
        return self.dX, self.dW

    def grad_input_mvue_weight(self, dY, step: int = 0, tensor_id_w: int | None = None):
        """Ablation (Sec. 5.1, the variant the paper rejects): grad_X = dY MVUE(S(W)^T)^T on sparse tensor cores.

        The sparsified operand must be 2:4 along the contraction dim O, so MVUE runs on w~ viewed as [O, I]
        (groups of four consecutive rows), giving the compressed [I, O] operand; the product is then the
        forward-type call with dY as the K-major operand.  bf16 only.  Composed of existing calls.
        """
        assert not self.fp8
        c = self.ctx
        if not hasattr(self, "wt_vals"):
            self.wt_vals, self.wt_meta = c.alloc_compressed(self.I, self.O, B.BF16)
            self.wt_dense = torch.empty((self.O, self.I), dtype=torch.bfloat16, device=self.W.device)
        tid = self.tensor_id + (1 << 16) if tensor_id_w is None else tensor_id_w     # a stream of its own
        c.decompress(self.vals, self.meta, self.wt_dense)
        c.mvue_sparsify(self.wt_dense, self.seed, tid, step, self.wt_vals, self.wt_meta)
        c.linear_fwd(dY, self.wt_vals, self.wt_meta, self.dX)
        self.launches += 3
        return self.dX

    def grad_weight_and_input(self, dY, side_ctx: B.Context, side_stream: torch.cuda.Stream):
        """grad_W on `side_stream` (through `side_ctx`: its own split-K workspace) while grad_X runs on the
        current stream: the two products are independent once MVUE has run, and the tail, second split-K pass
        and ramp-up of one overlap the other.  Both are complete in current-stream order on return."""
        main = torch.cuda.current_stream()
        side_stream.wait_stream(main)
        with torch.cuda.stream(side_stream):
            saved, self.ctx = self.ctx, side_ctx
            try:
                self.grad_weight()
            finally:
                self.ctx = saved
        self.grad_input(dY)
        main.wait_stream(side_stream)
        return self.dX, self.dW

    # (2b.1) MVUE(dY^T): 2:4 along tokens, compressed and transposed for the grad_W product
    def sparsify_grad(self, dY, step: int = 0, token_offset: int = 0):
        c = self.ctx
        if self.fp8:
            self._m("amax_g")
            c.amax(dY, self.amax[2:3])
            self.launches += 1
        self._m("mvue_sparsify")
        c.mvue_sparsify(dY, self.seed, self.tensor_id, step, self.gvals, self.gmeta,
                        dense_q_out=self.dYq if self.fp8 else None, g_amax_dev=self._amax(2),
                        token_offset=token_offset, counter_cols=self.counter_cols)
        self.launches += 1

    # (2b.2) grad_W = MVUE(dY^T) X, sparse
    def grad_weight(self):
        self._m("linear_bwd_weight")
        self.ctx.linear_bwd_weight(self.gvals, self.gmeta, self.Xq if self.fp8 else self.X, self.dW,
                                   g_amax_dev=self._amax(2), x_amax_dev=self._amax(0))
        self.launches += 1
        return self.dW

    # (2b.3) grad_X = dY w~, dense; w~ from the compressed operand unless a dense copy is kept
    def grad_input(self, dY, dx_amax_out=None):
        g = self.dYq if self.fp8 else dY
        self._m("linear_bwd_input")
        if self.w_dense is not None:
            self.ctx.linear_bwd_input(g, self.w_dense, self.dX, g_amax_dev=self._amax(2), w_amax_dev=self._amax(1),
                                      dx_amax_out_dev=dx_amax_out)
        else:
            self.ctx.linear_bwd_input(g, None, self.dX, g_amax_dev=self._amax(2), w_amax_dev=self._amax(1),
                                      vals=self.vals, meta=self.meta, dx_amax_out_dev=dx_amax_out)
        self.launches += 1
        return self.dX


class SsteLinearPadded:
    """An S-STE linear of ANY shape (W[O, I], T tokens), run on zero-padded copies.

    The library's kernels want multiples of 128.  Zero groups are fixed points of the projection (Eq. 4) and of
    the MVUE rule and add nothing to beta, to an amax or to a product, so padding W, X and dY with zeros and
    cropping Y, dX and dW gives the unpadded results; the MVUE counter runs over the unpadded column count.
    The pad and crop passes are library kernels too (sste_pad_2d / sste_crop_2d).
    """

    def __init__(self, ctx: B.Context, O: int, I: int, T: int, **kw):
        self.ctx, self.O, self.I, self.T = ctx, O, I, T
        self.Op, self.Ip, self.Tp = B.padded_dim(O), B.padded_dim(I), B.padded_dim(T)
        dev = f"cuda:{ctx.device}"
        bf = dict(dtype=torch.bfloat16, device=dev)
        self.Wp = torch.empty((self.Op, self.Ip), **bf)
        self.Xp = torch.empty((self.Tp, self.Ip), **bf)
        self.dYp = torch.empty((self.Tp, self.Op), **bf)
        self.inner = SsteLinear(ctx, self.Wp, self.Tp, counter_cols=O, **kw)
        self.Y = torch.empty((T, O), **bf)
        self.dX = torch.empty((T, I), **bf)
        self.dW = torch.empty((O, I), **bf)

    @property
    def beta(self):
        return self.inner.beta

    def set_weight(self, W):
        self.ctx.pad_2d(W, self.Wp)

    def init_beta(self):
        self.inner.init_beta()

    def prune(self):
        self.inner.prune()

    def forward(self, X):
        self.ctx.pad_2d(X, self.Xp)
        self.inner.forward(self.Xp)
        self.ctx.crop_2d(self.inner.Y, self.Y)
        return self.Y

    def backward(self, dY, step: int = 0):
        self.ctx.pad_2d(dY, self.dYp)
        self.inner.backward(self.dYp, step=step)
        self.ctx.crop_2d(self.inner.dX, self.dX)
        self.ctx.crop_2d(self.inner.dW, self.dW)
        return self.dX, self.dW
