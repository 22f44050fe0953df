"""Config 3: a small decoder-only transformer (6 layers, d_model 512, 8 heads, MLP 2048, pre-RMSNorm, vocab
32768, 64 sequences of 256 tokens, bf16, random init) as a harness around the library.

The harness is plain PyTorch and only produces what a training step would hand to the library: for every
linear layer the activations X entering it and the cotangents dY of its output, from the loss
sum_b (1/T) sum_t CE (so grad_scale = 1).  The library then computes sum_b G_b and sum_b G_b^2 per layer
and takes a MicroAdam step with the per-example squares as preconditioner; the oracle recomputes both
from the captured bf16 (X, dY) on sampled output rows and columns (it does not re-derive the model).
"""
import numpy as np
import pytest
import torch
import torch.nn as nn
import torch.nn.functional as F

import oracle
import paper_2510_00236_b200 as pe
from paper_2510_00236_b200 import inputs
from parity_util import FROB_TOL, boundary_and_random, rel_frob

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
D, HEADS, MLP, VOCAB, LAYERS, T, B = 512, 8, 2048, 32768, 6, 256, 64


class RMSNorm(nn.Module):
    def __init__(self, d):
        super().__init__()
        self.g = nn.Parameter(torch.ones(d))

    def forward(self, x):
        return x * torch.rsqrt(x.float().pow(2).mean(-1, keepdim=True) + 1e-6).to(x.dtype) * self.g


class Block(nn.Module):
    def __init__(self):
        super().__init__()
        self.n1, self.n2 = RMSNorm(D), RMSNorm(D)
        self.qkv, self.proj = nn.Linear(D, 3 * D, bias=False), nn.Linear(D, D, bias=False)
        self.up, self.down = nn.Linear(D, MLP, bias=False), nn.Linear(MLP, D, bias=False)

    def forward(self, x):
        b, t, _ = x.shape
        q, k, v = self.qkv(self.n1(x)).view(b, t, 3, HEADS, D // HEADS).permute(2, 0, 3, 1, 4)
        a = F.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(1, 2).reshape(b, t, D)
        x = x + self.proj(a)
        return x + self.down(F.gelu(self.up(self.n2(x))))


class Decoder(nn.Module):
    def __init__(self):
        super().__init__()
        self.emb, self.pos = nn.Embedding(VOCAB, D), nn.Embedding(T, D)
        self.blocks = nn.ModuleList(Block() for _ in range(LAYERS))
        self.norm, self.unembed = RMSNorm(D), nn.Linear(D, VOCAB, bias=False)

    def forward(self, ids):
        x = self.emb(ids) + self.pos(torch.arange(ids.shape[1], device=ids.device))
        for blk in self.blocks:
            x = blk(x)
        return self.unembed(self.norm(x))


def _capture(model, ids):
    """One forward/backward; returns {layer name: (X, dY, weight)} for every nn.Linear."""
    got, hooks = {}, []
    for name, mod in model.named_modules():
        if isinstance(mod, nn.Linear):
            def fwd(m, inp, out, name=name):
                got[name] = [inp[0].detach().contiguous(), None, m.weight]
                out.register_hook(lambda g, name=name: got[name].__setitem__(1, g.detach().contiguous()))
            hooks.append(mod.register_forward_hook(fwd))
    logits = model(ids[:, :-1])
    ce = F.cross_entropy(logits.float().reshape(-1, VOCAB), ids[:, 1:].reshape(-1), reduction="none")
    loss = ce.view(ids.shape[0], -1).mean(1).sum()          # sum over examples of the per-sequence mean
    loss.backward()
    for h in hooks:
        h.remove()
    return got


def test_config3_every_linear_layer_and_microadam_step():
    torch.manual_seed(inputs.BASE_SEED + 3)
    model = Decoder().to(DEV).to(torch.bfloat16)
    ids = torch.randint(0, VOCAB, (B, T + 1), generator=torch.Generator().manual_seed(inputs.BASE_SEED + 3)).to(DEV)
    layers = _capture(model, ids)
    assert len(layers) == 4 * LAYERS + 1
    kw = dict(lr=1e-3, beta1=0.9, beta2=0.999, eps=1e-8, step=1)
    worst = 0.0
    for name, (X, dY, W) in layers.items():
        d_out, d_in = W.shape
        assert X.dtype == torch.bfloat16 and dY.dtype == torch.bfloat16
        assert X.shape == (B, T, d_in) and dY.shape == (B, T, d_out)
        mean = torch.full((d_out, d_in), float("nan"), device=DEV)
        sq = torch.full((d_out, d_in), float("nan"), device=DEV)
        pe.pe_linear_stats(X, dY, "square", mean, sq)
        assert pe.pe_last_path() == pe.PATH_TENSOR
        theta = W.detach().float().contiguous()
        theta0 = theta.clone()
        m, v = torch.zeros_like(theta), torch.zeros_like(theta)
        pe.microadam_step(theta, m, v, mean, sq, B, **kw)
        torch.cuda.synchronize()
        # the ordinary weight gradient autograd computed must be sum_b G_b (bf16-rounded by autograd)
        g_auto = W.grad.float()
        assert rel_frob((mean - g_auto).cpu().numpy(), np.zeros(1)) <= 2e-2 * float(g_auto.norm())
        # oracle on sampled rows x columns of this layer, from the captured bf16 operands
        rows = boundary_and_random(d_out, 12, 31)
        cols = boundary_and_random(d_in, 12, 32)
        sub = inputs.gather_columns(inputs.LayerInputs(name, X, dY), rows, cols)
        st = oracle.linear_stats(inputs.to_numpy_bits(sub.X), inputs.to_numpy_bits(sub.dY))
        pick = lambda a: a.cpu().numpy()[np.asarray(rows)][:, np.asarray(cols)]
        e_mean, e_sq = rel_frob(pick(mean), st.sum_g), rel_frob(pick(sq), st.sum_g2)
        assert e_mean <= FROB_TOL and e_sq <= FROB_TOL, (name, e_mean, e_sq)
        th_ref, m_ref, v_ref = oracle.microadam_step(pick(theta0), np.zeros((len(rows), len(cols))), np.zeros((len(rows), len(cols))),
                                                     st.sum_g, st.sum_g2, B, **kw)
        e_upd = rel_frob(pick(theta) - pick(theta0), th_ref - pick(theta0).astype(np.float64))
        assert e_upd <= FROB_TOL, (name, e_upd)
        assert rel_frob(pick(v), v_ref) <= FROB_TOL and rel_frob(pick(m), m_ref) <= FROB_TOL
        # the same step with the update inside the statistics kernel and no statistic buffers at all
        theta_f, m_f, v_f = theta0.clone(), torch.zeros_like(theta), torch.zeros_like(theta)
        pe.pe_linear_microadam_step(X, dY, theta_f, m_f, v_f, **kw)
        torch.cuda.synchronize()
        e_fused = rel_frob(pick(theta_f) - pick(theta0), th_ref - pick(theta0).astype(np.float64))
        assert e_fused <= FROB_TOL, (name, e_fused)
        assert rel_frob(pick(v_f), v_ref) <= FROB_TOL and rel_frob(pick(m_f), m_ref) <= FROB_TOL
        worst = max(worst, e_mean, e_sq, e_upd, e_fused)
    assert pe.pe_get_async_status(DEV) == (0, 0)
    print("config3: 25 linear layers, worst relative Frobenius error", worst)
