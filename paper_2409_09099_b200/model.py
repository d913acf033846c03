"""A GPT-2-124M-shaped decoder whose linear layers all run through libsste (a harness, not part of the hot path).

12 blocks of d = 768, 12 heads, FFN 3072, sequence 1024, vocabulary 50257.  The 48 linears (per block: qkv
[2304, 768], attention output [768, 768], fc1 [3072, 768], fc2 [768, 3072]) are S-STE linears: every training
step prunes the dense weight (Eq. 4, beta frozen after the first step, Sec. 4.2), runs forward and backward
with the sparse weight (Sec. 5.1) and hands grad_W to the optimiser unchanged (straight-through estimator,
Eq. 3).  Embeddings, layer norms, attention, GELU, the tied output projection, the loss and AdamW are stock
torch operations: they only produce the activations and gradients the S-STE linears consume.

Used by the config-4 test and by ``bench.py --config 4``; `on_call` lets a test inspect every libsste call.
"""
from __future__ import annotations

import torch
import torch.nn.functional as F

from . import binding as B
from .layer import SsteLinear


class _SsteFn(torch.autograd.Function):
    """Y = X S(W)^T through libsste; the gradient with respect to the fp32 master weight is grad_W (Eq. 3)."""

    @staticmethod
    def forward(ctx, x, w_master, owner):
        ctx.owner = owner
        lin = owner.lin
        owner.t0 = owner.model._tick()
        y = lin.forward(x)
        owner.model._tock(owner.t0)
        owner.x = x
        return y.detach()          # a fresh tensor object over the layer's output buffer

    @staticmethod
    def backward(ctx, dy):
        owner = ctx.owner
        lin, model = owner.lin, owner.model
        dy = dy.contiguous()
        t0 = model._tick()
        dx, dw = lin.backward(dy, step=model.step_index)
        model._tock(t0)
        if model.on_call is not None:
            model.on_call(owner.index, model.step_index, lin, owner.x, dy)
        return dx, dw.float(), None


class SparseLinear:
    """fp32 master weight + bias (torch parameters) in front of one SsteLinear working on a bf16 copy."""

    def __init__(self, model, index, O, I, T, std, gen):
        dev = model.device
        self.model, self.index = model, index
        self.w = torch.nn.Parameter(torch.randn((O, I), device=dev, generator=gen) * std)
        self.b = torch.nn.Parameter(torch.zeros(O, device=dev))
        self.w16 = torch.empty((O, I), dtype=torch.bfloat16, device=dev)
        self.lin = SsteLinear(model.ctx, self.w16, T, tensor_id=index, seed=model.seed)
        self.beta_launches = 0
        self.x = None

    def refresh(self):
        """Start of a training step: the dense weight as bf16, beta in the first step only, then the projection."""
        self.w16.copy_(self.w.detach())
        t0 = self.model._tick()
        if not self.lin.beta_ready:
            self.lin.init_beta()
            self.beta_launches += 1
        self.lin.prune()
        self.model._tock(t0)

    def __call__(self, x):
        return _SsteFn.apply(x, self.w, self) + self.b.to(torch.bfloat16)


class SsteGpt2:
    def __init__(self, ctx: B.Context, n_layer=12, d=768, n_head=12, d_ff=3072, seq=1024, batch=8, vocab=50257,
                 seed=4, lr=3e-4):
        self.ctx, self.device, self.seed = ctx, f"cuda:{ctx.device}", seed
        self.n_layer, self.d, self.n_head, self.seq, self.batch, self.vocab = n_layer, d, n_head, seq, batch, vocab
        T = batch * seq
        gen = torch.Generator(device=self.device).manual_seed(seed)
        self.wte = torch.nn.Parameter(torch.randn((vocab, d), device=self.device, generator=gen) * 0.02)
        self.wpe = torch.nn.Parameter(torch.randn((seq, d), device=self.device, generator=gen) * 0.02)
        self.linears, self.norms = [], []
        for l in range(n_layer):
            for O, I in ((3 * d, d), (d, d), (d_ff, d), (d, d_ff)):
                self.linears.append(SparseLinear(self, len(self.linears), O, I, T, 0.02, gen))
            self.norms.append([torch.nn.Parameter(torch.ones(d, device=self.device)),
                               torch.nn.Parameter(torch.zeros(d, device=self.device)),
                               torch.nn.Parameter(torch.ones(d, device=self.device)),
                               torch.nn.Parameter(torch.zeros(d, device=self.device))])
        self.ln_f = [torch.nn.Parameter(torch.ones(d, device=self.device)),
                     torch.nn.Parameter(torch.zeros(d, device=self.device))]
        params = [self.wte, self.wpe] + [p for s in self.linears for p in (s.w, s.b)] + \
                 [p for n in self.norms for p in n] + self.ln_f
        self.opt = torch.optim.AdamW(params, lr=lr, weight_decay=0.0)
        self.step_index = 0
        self.on_call = None
        self._timing = None        # list of (start, end) CUDA events of the libsste calls of one step

    # ---- time spent inside libsste (CUDA events around its calls, when enabled)
    def _tick(self):
        if self._timing is None:
            return None
        e = torch.cuda.Event(enable_timing=True)
        e.record()
        return e

    def _tock(self, e0):
        if e0 is not None:
            e1 = torch.cuda.Event(enable_timing=True)
            e1.record()
            self._timing.append((e0, e1))

    def flops_per_step(self):
        """dense-equivalent flops of the S-STE linears: 6 T I O each (forward, grad_W, grad_X)."""
        return sum(6.0 * self.batch * self.seq * s.lin.O * s.lin.I for s in self.linears)

    def loss(self, tokens, targets):
        Bsz, S, d, H = self.batch, self.seq, self.d, self.n_head
        x = (self.wte[tokens] + self.wpe[None, :S]).to(torch.bfloat16).view(Bsz * S, d)
        for l in range(self.n_layer):
            qkv_l, proj_l, fc1_l, fc2_l = self.linears[4 * l: 4 * l + 4]
            g1, b1, g2, b2 = self.norms[l]
            h = F.layer_norm(x.float(), (d,), g1, b1).to(torch.bfloat16)
            q, k, v = qkv_l(h).view(Bsz, S, 3, H, d // H).permute(2, 0, 3, 1, 4)
            a = F.scaled_dot_product_attention(q, k, v, is_causal=True)
            a = a.transpose(1, 2).reshape(Bsz * S, d).contiguous()
            x = x + proj_l(a)
            h = F.layer_norm(x.float(), (d,), g2, b2).to(torch.bfloat16)
            x = x + fc2_l(F.gelu(fc1_l(h), approximate="tanh").contiguous())
        h = F.layer_norm(x.float(), (d,), *self.ln_f).to(torch.bfloat16)
        logits = h @ self.wte.to(torch.bfloat16).t()            # tied output projection, dense
        return F.cross_entropy(logits.float(), targets.view(-1))

    def train_step(self, tokens, targets, time_libsste=False):
        """Prune every linear, forward, backward, optimiser step.  Returns (loss, seconds in libsste or None)."""
        self._timing = [] if time_libsste else None
        for s in self.linears:
            s.refresh()
        self.opt.zero_grad(set_to_none=True)
        loss = self.loss(tokens, targets)
        loss.backward()
        self.opt.step()
        inside = None
        if time_libsste:
            torch.cuda.synchronize()
            inside = sum(a.elapsed_time(b) for a, b in self._timing) * 1e-3
            self._timing = None
        self.step_index += 1
        return loss.detach(), inside


def synthetic_batch(model: SsteGpt2, seed: int):
    """Uniform token ids in [0, vocab) and next-token targets (a fixed synthetic batch)."""
    gen = torch.Generator(device=model.device).manual_seed(seed)
    ids = torch.randint(0, model.vocab, (model.batch, model.seq + 1), device=model.device, generator=gen)
    return ids[:, :-1].contiguous(), ids[:, 1:].contiguous()

