"""AGZO on a transformer block as a user would run it: the forward is plain torch, forward hooks
copy the inputs of the seven linear layers into persistent bf16 buffers during the unperturbed
forward (Algorithm 2, step 1), and agzo_step does the rest.  q/k/v read one buffer and gate/up
another, so the library serves each of those groups with one sweep over the activations.

What is checked is what must hold whatever the model: the step's scalar g is the directional
derivative along the direction the library applied, so for a small step the loss falls by
lr * g^2 to first order (Section 3.3: the update is -eta * g * Delta with g = <grad f, Delta> + O(mu)).
"""
import numpy as np
import pytest
import torch

from paper_2601_17261_b200 import binding as B

from gpu_helpers import DEV

pytestmark = pytest.mark.gpu

HID, HEADS, KV_HEADS, HEAD_DIM, INTER, BATCH, SEQ = 256, 4, 2, 64, 512, 2, 128


def _rms(x):
    return x / torch.sqrt((x * x).mean(-1, keepdim=True) + 1e-6)


class Block:
    """Pre-norm attention + gated MLP with grouped-query attention; weights are the caller's tensors."""
    names = ["q", "k", "v", "o", "gate", "up", "down"]

    def __init__(self, dtype, seed=0):
        g = torch.Generator(device="cpu").manual_seed(seed)
        shapes = {"q": (HEADS * HEAD_DIM, HID), "k": (KV_HEADS * HEAD_DIM, HID), "v": (KV_HEADS * HEAD_DIM, HID),
                  "o": (HID, HEADS * HEAD_DIM), "gate": (INTER, HID), "up": (INTER, HID), "down": (HID, INTER)}
        self.W = {n: (torch.randn(s, generator=g) / np.sqrt(s[1])).to(DEV).to(dtype) for n, s in shapes.items()}
        m = BATCH * SEQ
        # inputs of the linear layers, written by the forward when `capture` is set
        self.X = {"qkv": torch.zeros(m, HID, dtype=torch.bfloat16, device=DEV),
                  "o": torch.zeros(m, HEADS * HEAD_DIM, dtype=torch.bfloat16, device=DEV),
                  "mlp": torch.zeros(m, HID, dtype=torch.bfloat16, device=DEV),
                  "down": torch.zeros(m, INTER, dtype=torch.bfloat16, device=DEV)}
        self.x0 = torch.randn(BATCH, SEQ, HID, generator=g).to(DEV).double()
        self.target = torch.randn(BATCH, SEQ, HID, generator=g).to(DEV).double()

    def x_of(self, name):
        return self.X["qkv" if name in "qkv" else "mlp" if name in ("gate", "up") else name]

    def forward(self, capture=False):
        W = {n: w.double() for n, w in self.W.items()}
        x = self.x0
        h = _rms(x)
        if capture:
            self.X["qkv"].copy_(h.reshape(-1, HID))
        q = (h @ W["q"].t()).view(BATCH, SEQ, HEADS, HEAD_DIM).transpose(1, 2)
        k = (h @ W["k"].t()).view(BATCH, SEQ, KV_HEADS, HEAD_DIM).transpose(1, 2)
        v = (h @ W["v"].t()).view(BATCH, SEQ, KV_HEADS, HEAD_DIM).transpose(1, 2)
        k = k.repeat_interleave(HEADS // KV_HEADS, dim=1)
        v = v.repeat_interleave(HEADS // KV_HEADS, dim=1)
        att = (q @ k.transpose(-1, -2)) / np.sqrt(HEAD_DIM)
        att = att.masked_fill(torch.triu(torch.ones(SEQ, SEQ, device=DEV, dtype=torch.bool), 1), float("-inf"))
        a = (torch.softmax(att, -1) @ v).transpose(1, 2).reshape(BATCH, SEQ, HEADS * HEAD_DIM)
        if capture:
            self.X["o"].copy_(a.reshape(-1, HEADS * HEAD_DIM))
        x = x + a @ W["o"].t()
        h2 = _rms(x)
        if capture:
            self.X["mlp"].copy_(h2.reshape(-1, HID))
        act = torch.nn.functional.silu(h2 @ W["gate"].t()) * (h2 @ W["up"].t())
        if capture:
            self.X["down"].copy_(act.reshape(-1, INTER))
        x = x + act @ W["down"].t()
        return ((x - self.target) ** 2).mean()


@pytest.mark.parametrize("dtype,r", [(torch.float32, 4), (torch.bfloat16, 8)])
def test_agzo_steps_on_a_transformer_block(dtype, r):
    blk = Block(dtype)
    Vs = {n: torch.zeros(r, blk.W[n].shape[1], device=DEV) for n in Block.names}
    layers = [B.make_layer(W=blk.W[n], X=blk.x_of(n), V=Vs[n], r=r, layer_id=i) for i, n in enumerate(Block.names)]
    assert layers[0].X == layers[1].X == layers[2].X and layers[4].X == layers[5].X     # shared inputs
    losses = torch.zeros(2, dtype=torch.float64, device=DEV)
    ghat = torch.zeros(1, device=DEV)
    calls = []

    def loss_fn(phase, slot, stream):
        calls.append(phase)
        losses[slot] = blk.forward(capture=(phase == 0))

    ctx = B.agzo_create(layers, 0)
    try:
        eps, lr = 1e-3, 2e-3
        f_prev = float(blk.forward())
        ratios = []
        for step in range(6):
            B.agzo_step(ctx, layers, seed=100 + step, eps=eps, lr=lr, K=3, mode=0, loss_fn=loss_fn,
                        d_losses2=losses, d_ghat=ghat)
            assert B.agzo_poll(ctx) == B.AGZO_OK
            g = float(ghat)
            f_now = float(blk.forward())
            if dtype == torch.float32 and abs(g) > 1e-2:
                ratios.append((f_prev - f_now) / (lr * g * g))       # first order: 1
            f_prev = f_now
        assert calls[:3] == [0, 1, 2] and len(calls) == 18
        for n in Block.names:                                         # every V is an orthonormal basis
            V = Vs[n].double()
            assert float((V @ V.t() - torch.eye(r, device=DEV, dtype=torch.float64)).abs().max()) <= 1e-5
        if dtype == torch.float32:
            assert ratios and all(0.7 <= x <= 1.3 for x in ratios), ratios
    finally:
        B.agzo_destroy(ctx)
