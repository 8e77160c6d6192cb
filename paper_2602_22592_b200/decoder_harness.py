"""A LLaMA-style decoder whose every projection is a pQuant linear: the harness around the C entry points for the
"whole training step" workload (24 layers, hidden 2048, 16 heads, FFN 5632, RMSNorm, RoPE, vocabulary 32000 at
full size).

Only the projections are the product: each one is `pq_pack_weights` + `pq_linear_forward` in the forward pass and
`pq_linear_backward` in the backward pass, reached through a torch.autograd.Function that marshals pointers and
nothing else.  Everything between the projections -- embedding, RMSNorm, rotary embedding, attention, SiLU gating,
LM head, cross-entropy -- is ordinary torch and lies outside the library's boundary; it is here so that the
projections run in the order, on the activations and beside the foreign kernels a real QAT step gives them.

CUDA events around every pq_* call let the caller report the pQuant-linear time of a step apart from the rest.
"""
from __future__ import annotations

import math

import torch
import torch.nn.functional as F

from . import binding as pqb


class _Workspaces:
    """Forward / backward / pack workspaces shared by all linears of one model (calls are serial on one stream)."""

    def __init__(self, device):
        self.dev = device
        self.fwd = self.bwd = self.pack = None

    def reserve(self, desc):
        def grow(buf, n):
            return buf if buf is not None and buf.numel() >= n else torch.empty(max(n, 16), dtype=torch.uint8, device=self.dev)
        self.fwd = grow(self.fwd, pqb.pq_workspace_bytes(desc, pqb.PQ_PHASE_FWD))
        self.bwd = grow(self.bwd, pqb.pq_workspace_bytes(desc, pqb.PQ_PHASE_BWD))
        self.pack = grow(self.pack, pqb.pq_workspace_bytes(desc, pqb.PQ_PHASE_PACK))


class Timer:
    """Sums the device time of the pq_* calls of a step: one event pair per call, read after the step."""

    def __init__(self):
        self.pairs = []
        self.enabled = False

    def begin(self):
        if not self.enabled:
            return None
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        self.pairs.append((a, b))
        return b

    @staticmethod
    def end(b):
        if b is not None:
            b.record()

    def total_ms(self):
        """Call after a synchronise.  Clears the recorded pairs."""
        t = sum(a.elapsed_time(b) for a, b in self.pairs)
        self.pairs = []
        return t


class _PQLinearFn(torch.autograd.Function):
    """x [T,K] bf16 -> y [T,N] bf16 through the C ABI.  Parameter gradients are not returned to autograd: the
    library overwrites the module's gradient buffers (dW, dA, dB, dWr, dalpha, dbeta), which is what the ABI
    promises; accumulation over micro-batches would be the optimiser's business."""

    @staticmethod
    def forward(ctx, x, mod):
        ctx.mod = mod
        x = x.contiguous()
        ctx.save_for_backward(x)
        return mod._forward(x)

    @staticmethod
    def backward(ctx, dy):
        (x,) = ctx.saved_tensors
        return ctx.mod._backward(x, dy.contiguous()), None


class PQLinearModule:
    """One pQuant linear (Eq. 10-11, Sec. 3.3) of a model: latent fp32 W, bf16 experts A, B, router Wr, scalar feature
    scales; `saved` is its own (it lives from forward to backward), workspaces are the model's."""

    def __init__(self, T, K, N, r, E, ws: _Workspaces, timer: Timer, gen, device, name=""):
        self.T, self.K, self.N, self.r, self.E, self.name = T, K, N, r, (E if r > 0 else 0), name
        self.ws, self.timer = ws, timer
        self.desc = pqb.make_desc(T, K, N, r, self.E, 1, False)
        ws.reserve(self.desc)
        dev = device
        std = 0.02
        self.W = torch.randn((N, K), generator=gen, device=dev, dtype=torch.float32) * std
        Ee = max(self.E, 1)
        if r > 0:
            self.A = (torch.randn((Ee, r, K), generator=gen, device=dev) * std).to(torch.bfloat16)
            self.B = (torch.randn((Ee, N, r), generator=gen, device=dev) * std).to(torch.bfloat16)
            self.Wr = (torch.randn((Ee, K), generator=gen, device=dev) * std).to(torch.bfloat16) if Ee > 1 else None
            self.dA = torch.empty((Ee, r, K), dtype=torch.float32, device=dev)
            self.dB = torch.empty((Ee, N, r), dtype=torch.float32, device=dev)
            self.dWr = torch.empty((Ee, K), dtype=torch.float32, device=dev) if Ee > 1 else None
        else:
            self.A = self.B = self.Wr = self.dA = self.dB = self.dWr = None
        self.alpha = torch.full((1,), 2.0, device=dev)     # the paper's initial feature scales (Sec. 3.2)
        self.beta = torch.full((1,), 0.2, device=dev)
        self.dalpha = torch.empty(1, dtype=torch.float32, device=dev)
        self.dbeta = torch.empty(1, dtype=torch.float32, device=dev)
        self.dW = torch.empty((N, K), dtype=torch.float32, device=dev)
        self.w_bits = torch.empty((N, K // 32), dtype=torch.int32, device=dev)
        self.w_s8 = torch.empty((N, K), dtype=torch.int8, device=dev)
        self.w_scales = torch.empty(2, dtype=torch.float32, device=dev)
        self.saved = torch.empty(pqb.pq_saved_bytes(self.desc), dtype=torch.uint8, device=dev)
        self.capture = None        # set to a dict by tests: receives x, y, dy, dx of the next call

    def __call__(self, x):
        return _PQLinearFn.apply(x, self)

    def _forward(self, x):
        assert x.shape == (self.T, self.K) and x.dtype == torch.bfloat16
        y = torch.empty((self.T, self.N), dtype=torch.bfloat16, device=x.device)
        ev = self.timer.begin()
        # QAT re-quantises the latent weights in every forward pass
        pqb.pq_pack_weights(self.desc, self.W, self.w_bits, self.w_s8, self.w_scales, self.ws.pack)
        pqb.pq_linear_forward(self.desc, x, self.w_bits, self.w_s8, self.w_scales, self.A, self.B, self.Wr, self.alpha, self.beta, y,
                              self.saved, self.ws.fwd)
        self.timer.end(ev)
        if self.capture is not None:
            self.capture.update(x=x.detach().clone(), y=y.detach().clone())
        return y

    def _backward(self, x, dy):
        dx = torch.empty((self.T, self.K), dtype=torch.bfloat16, device=x.device)
        ev = self.timer.begin()
        pqb.pq_linear_backward(self.desc, dy, x, self.w_s8, self.w_scales, self.A, self.B, self.Wr, self.alpha, self.beta, self.saved,
                               dx, self.dW, self.dA, self.dB, self.dWr, self.dalpha, self.dbeta, self.ws.bwd)
        self.timer.end(ev)
        if self.capture is not None:
            self.capture.update(dy=dy.detach().clone(), dx=dx.detach().clone())
        return dx


def _rope_tables(seq, head_dim, device, base=10000.0):
    inv = 1.0 / (base ** (torch.arange(0, head_dim, 2, device=device, dtype=torch.float32) / head_dim))
    ang = torch.outer(torch.arange(seq, device=device, dtype=torch.float32), inv)     # [S, D/2]
    return ang.cos(), ang.sin()


def _apply_rope(x, cos, sin):
    # x [B, H, S, D]; rotate pairs (even, odd halves)
    d = x.shape[-1] // 2
    x1, x2 = x[..., :d].float(), x[..., d:].float()
    return torch.cat([x1 * cos - x2 * sin, x2 * cos + x1 * sin], dim=-1).to(x.dtype)


class PQDecoder:
    """The decoder.  `attn_hp=False` makes the four attention projections pure 1-bit linears (r = 0), the form the
    paper gives its attention blocks (Sec. 3); True gives them the same routed HP branch as the MLP projections."""

    def __init__(self, layers=24, hidden=2048, heads=16, ffn=5632, vocab=32000, batch=4, seq=2048, r=128, E=8, attn_hp=True,
                 device="cuda:0", seed=3):
        self.dev = torch.device(device)
        self.layers, self.hidden, self.heads, self.ffn, self.vocab, self.batch, self.seq = layers, hidden, heads, ffn, vocab, batch, seq
        self.head_dim = hidden // heads
        gen = torch.Generator(device=self.dev)
        gen.manual_seed(seed)
        T = batch * seq
        self.T = T
        self.ws = _Workspaces(self.dev)
        self.timer = Timer()
        mk = lambda K, N, rr, name: PQLinearModule(T, K, N, rr, E, self.ws, self.timer, gen, self.dev, name)
        ra = r if attn_hp else 0
        self.blocks = []
        for i in range(layers):
            blk = dict(q=mk(hidden, hidden, ra, f"L{i}.q"), k=mk(hidden, hidden, ra, f"L{i}.k"), v=mk(hidden, hidden, ra, f"L{i}.v"),
                       o=mk(hidden, hidden, ra, f"L{i}.o"), gate=mk(hidden, ffn, r, f"L{i}.gate"), up=mk(hidden, ffn, r, f"L{i}.up"),
                       down=mk(ffn, hidden, r, f"L{i}.down"),
                       norm1=torch.ones(hidden, device=self.dev, dtype=torch.bfloat16, requires_grad=True),
                       norm2=torch.ones(hidden, device=self.dev, dtype=torch.bfloat16, requires_grad=True))
            self.blocks.append(blk)
        self.embed = (torch.randn((vocab, hidden), generator=gen, device=self.dev) * 0.02).to(torch.bfloat16).requires_grad_(True)
        self.head = (torch.randn((vocab, hidden), generator=gen, device=self.dev) * 0.02).to(torch.bfloat16).requires_grad_(True)
        self.norm_f = torch.ones(hidden, device=self.dev, dtype=torch.bfloat16, requires_grad=True)
        self.cos, self.sin = _rope_tables(seq, self.head_dim, self.dev)
        self.gen = gen

    def linears(self):
        for blk in self.blocks:
            for k in ("q", "k", "v", "o", "gate", "up", "down"):
                yield blk[k]

    def random_batch(self):
        ids = torch.randint(0, self.vocab, (self.batch, self.seq), generator=self.gen, device=self.dev)
        tgt = torch.randint(0, self.vocab, (self.batch, self.seq), generator=self.gen, device=self.dev)
        return ids, tgt

    def _torch_params(self):
        ps = [self.embed, self.head, self.norm_f]
        for blk in self.blocks:
            ps += [blk["norm1"], blk["norm2"]]
        return ps

    def step(self, ids, tgt):
        """One forward + backward (no optimiser).  Returns the loss tensor."""
        for p in self._torch_params():
            p.grad = None
        B, S, H, D = self.batch, self.seq, self.heads, self.head_dim
        x = F.embedding(ids, self.embed).view(B * S, self.hidden)
        for blk in self.blocks:
            h = F.rms_norm(x, (self.hidden,), blk["norm1"], 1e-5)
            q = blk["q"](h).view(B, S, H, D).transpose(1, 2)
            k = blk["k"](h).view(B, S, H, D).transpose(1, 2)
            v = blk["v"](h).view(B, S, H, D).transpose(1, 2)
            q, k = _apply_rope(q, self.cos, self.sin), _apply_rope(k, self.cos, self.sin)
            a = F.scaled_dot_product_attention(q, k, v, is_causal=True)
            a = a.transpose(1, 2).reshape(B * S, self.hidden)
            x = x + blk["o"](a)
            h = F.rms_norm(x, (self.hidden,), blk["norm2"], 1e-5)
            m = F.silu(blk["gate"](h)) * blk["up"](h)
            x = x + blk["down"](m)
        x = F.rms_norm(x, (self.hidden,), self.norm_f, 1e-5)
        logits = x @ self.head.t()
        loss = F.cross_entropy(logits.float(), tgt.view(-1))
        loss.backward()
        return loss.detach()

    def roofline_time_s(self, p_bf16, p_i8):
        """Sum over the linears of 2TNK / P_i8 + (4TNK + 6Tr(K+N)) / P_bf16."""
        t = 0.0
        for L in self.linears():
            tnk = L.T * L.N * L.K
            t += 2 * tnk / p_i8 + (4 * tnk + 6 * L.T * L.r * (L.K + L.N)) / p_bf16
        return t


def softmax_entropy_bound(vocab):
    """Loss of a uniform prediction, ln(vocab): what a randomly initialised model should be near."""
    return math.log(vocab)
