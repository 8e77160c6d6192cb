"""Buffer management around the C entry points for one pQuant linear layer.

Holds the device tensors (inputs, packed weights, saved activations, gradients,
workspaces) for a fixed shape and calls pq_pack_weights / pq_linear_forward /
pq_linear_backward on them.  No arithmetic happens here.
"""
from __future__ import annotations

import numpy as np
import torch

from . import binding as pqb


def _bf16(a, dev):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev).to(torch.bfloat16).contiguous()


def _f32(a, dev):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(dev).contiguous()


GUARD_BYTES = 4096      # canary band in front of and behind every guarded buffer
GUARD_BYTE = 0xA5


class PQLinear:
    """One decoupled linear layer of fixed shape on one CUDA device.

    guard=True puts a band of canary bytes in front of and behind every buffer the library writes
    (outputs, packed weights, the saved buffer, the workspaces); `check_guards()` then tells whether
    any kernel wrote outside the bytes it was given.  (torch's caching allocator rounds sizes up, so an
    overrun of an exact-size tensor would otherwise land in slack nobody looks at.)"""

    def __init__(self, T, K, N, r=0, E=0, scale_vector=False, device="cuda:0", training=True, dump_acc=False, guard=False,
                 fused_rmsnorm=False):
        self.dev = torch.device(device)
        self.T, self.K, self.N, self.r, self.E = T, K, N, r, (E if r > 0 else 0)
        self.scale_vector = scale_vector
        self.desc = pqb.make_desc(T, K, N, r, self.E, 1, scale_vector, fused_rmsnorm=fused_rmsnorm and training)
        self.fused_rmsnorm = fused_rmsnorm and training
        self.guard = guard
        self._guards = []
        self.w_bits = self._buf((N, K // 32), torch.int32)
        self.w_s8 = self._buf((N, K), torch.int8)
        self.w_scales = self._buf((2,), torch.float32)
        self.ws_pack = self._buf((pqb.pq_workspace_bytes(self.desc, pqb.PQ_PHASE_PACK),), torch.uint8)
        self.training = training
        if training:
            nb = pqb.pq_saved_bytes(self.desc)
            if nb == 0:
                raise pqb.PqError("pq_saved_bytes", pqb.PQ_ERR_SHAPE)
            self.saved = self._buf((nb,), torch.uint8)
            self.ws_fwd = self._buf((pqb.pq_workspace_bytes(self.desc, pqb.PQ_PHASE_FWD),), torch.uint8)
            self.ws_bwd = self._buf((max(16, pqb.pq_workspace_bytes(self.desc, pqb.PQ_PHASE_BWD)),), torch.uint8)
            self.Y = self._buf((T, N), torch.bfloat16)
            self.dX = self._buf((T, K), torch.bfloat16)
            self.dW = self._buf((N, K), torch.float32)
            ns = N if scale_vector else 1
            self.dalpha = self._buf((ns,), torch.float32)
            self.dbeta = self._buf((ns,), torch.float32)
            if r > 0:
                Ee = max(self.E, 1)
                self.dA = self._buf((Ee, r, K), torch.float32)
                self.dB = self._buf((Ee, N, r), torch.float32)
                self.dWr = self._buf((Ee, K), torch.float32) if Ee > 1 else None
            else:
                self.dA = self.dB = self.dWr = None
        else:
            # decode: T <= 16 tokens straight from the packed bits
            self.desc = pqb.make_desc(T, K, N, r, self.E, 1, scale_vector, dump_acc=dump_acc)
            nb = pqb.pq_workspace_bytes(self.desc, pqb.PQ_PHASE_DECODE)
            self.ws_decode = self._buf((max(nb, 16),), torch.uint8).zero_() if T <= 16 else None
            self.Y = self._buf((T, N), torch.bfloat16)
        self.X = self.W = self.A = self.B = self.Wr = self.alpha = self.beta = self.dY = None
        self.w_bits_il = self.B_il = None
        self.B8_il = None   # set by pack_decode_hp8(): decode then runs the INT8 high-precision branch

    # -- buffers --------------------------------------------------------------
    def _buf(self, shape, dtype):
        """A device buffer the library writes into; with guard=True carved out of a larger allocation
        whose first and last GUARD_BYTES hold the canary pattern."""
        if not self.guard:
            return torch.empty(shape, dtype=dtype, device=self.dev)
        n = 1
        for s in shape:
            n *= s
        nbytes = n * torch.empty(0, dtype=dtype).element_size()
        raw = torch.full((nbytes + 2 * GUARD_BYTES,), GUARD_BYTE, dtype=torch.uint8, device=self.dev)
        self._guards.append((raw, nbytes))
        return raw[GUARD_BYTES:GUARD_BYTES + nbytes].view(dtype).view(*shape)

    def check_guards(self) -> int:
        """Number of canary bytes that no longer hold the pattern (0 = nothing was written out of bounds)."""
        bad = 0
        for raw, nbytes in self._guards:
            bad += int((raw[:GUARD_BYTES] != GUARD_BYTE).sum()) + int((raw[GUARD_BYTES + nbytes:] != GUARD_BYTE).sum())
        return bad

    # -- data ---------------------------------------------------------------
    def load_case(self, case: dict):
        """Upload a dict produced by inputs.make_linear_case."""
        dev = self.dev
        self.X = _bf16(case["X"], dev)
        self.W = _f32(case["W"], dev)
        self.A = _bf16(case.get("A"), dev) if self.r > 0 else None
        self.B = _bf16(case.get("B"), dev) if self.r > 0 else None
        self.Wr = _bf16(case.get("Wr"), dev) if (self.r > 0 and self.E > 1) else None
        self.alpha = _f32(case["alpha"], dev)
        self.beta = _f32(case["beta"], dev)
        self.dY = _bf16(case.get("dY"), dev)
        return self

    # -- calls --------------------------------------------------------------
    stream_decode = True   # decode layers also get the streaming kernel's weight layout when they are packed

    def pack(self, bits_only=False):
        pqb.pq_pack_weights(self.desc, self.W, self.w_bits, None if bits_only else self.w_s8, self.w_scales, self.ws_pack)
        if not self.training and PQLinear.stream_decode and self.T <= 16 and (self.r == 0 or self.B is not None):
            self.pack_decode()

    def pack_decode(self):
        """Lay the packed bits and B out for the streaming decode kernel (after pack() and load_case()); decode() and
        decode_entry() then hand both layouts to the library.  Returns False when the shape has no such layout."""
        if self.r % 8:
            return False
        nb, nB = pqb.pq_decode_pack_bytes(self.desc)
        self.w_bits_il = self._buf((nb,), torch.uint8)
        self.B_il = self._buf((nB,), torch.uint8) if nB else None
        pqb.pq_pack_decode(self.desc, self.w_bits, self.B, self.w_bits_il, self.B_il)
        return True

    def pack_decode_hp8(self):
        """INT8 high-precision branch for decode: quantise the experts (pack_experts) and lay B8 out for the streaming
        kernel; decode() and decode_entry() then use it (needs pack_decode() too)."""
        self.pack_experts()
        self.B8_il = self._buf((pqb.pq_decode_pack_hp8_bytes(self.desc),), torch.uint8)
        pqb.pq_pack_decode_hp8(self.desc, self.B8, self.B8_il)

    def decode(self, X=None, Y=None):
        """Inference forward from the packed sign bits (w_s8 is not used).  With `norm_weight` set, X is the
        un-normalised activation and RMSNorm is fused in front of the quantiser (a batch of one)."""
        if getattr(self, "norm_weight", None) is not None or self.w_bits_il is not None:
            entry = list(self.decode_entry())
            if X is not None: entry[1] = X
            if Y is not None: entry[9] = Y
            items = pqb.make_decode_items([tuple(entry)])
            pqb.pq_decode_batch(items)
            return self.Y if Y is None else Y
        pqb.pq_linear_forward(self.desc, self.X if X is None else X, self.w_bits, None, self.w_scales, self.A, self.B, self.Wr,
                              self.alpha, self.beta, self.Y if Y is None else Y, None, self.ws_decode)
        return self.Y if Y is None else Y

    def decode_entry(self):
        """This layer's arguments as one entry for binding.make_decode_items."""
        return (self.desc, self.X, self.w_bits, self.w_scales, self.A, self.B, self.Wr, self.alpha, self.beta, self.Y, self.ws_decode,
                getattr(self, "norm_weight", None), getattr(self, "norm_eps", 0.0), self.w_bits_il, self.B_il,
                self.A8 if self.B8_il is not None else None, self.B8_il, self.hp_scales if self.B8_il is not None else None)

    def decode_view(self) -> dict:
        return pqb.pq_decode_view_init(self.desc, self.ws_decode)

    def forward(self, X=None, Y=None):
        if self.fused_rmsnorm:      # X is the un-normalised activation; norm_weight / norm_eps set by the caller
            pqb.pq_linear_forward_rms(self.desc, self.X if X is None else X, self.norm_weight, self.norm_eps, self.w_s8, self.w_scales,
                                      self.A, self.B, self.Wr, self.alpha, self.beta, self.Y if Y is None else Y, self.saved, self.ws_fwd)
            return self.Y if Y is None else Y
        pqb.pq_linear_forward(self.desc, self.X if X is None else X, self.w_bits, self.w_s8, self.w_scales, self.A, self.B,
                              self.Wr, self.alpha, self.beta, self.Y if Y is None else Y, self.saved, self.ws_fwd)
        return self.Y if Y is None else Y

    def pack_experts(self):
        """INT8 codes and scales of the expert matrices (Sec. 3.2), kept beside the bf16 originals."""
        Ee = max(self.E, 1)
        if getattr(self, "A8", None) is None:
            self.A8 = self._buf((Ee, self.r, self.K), torch.int8)
            self.B8 = self._buf((Ee, self.N, self.r), torch.int8)
            self.hp_scales = self._buf((Ee, 2), torch.float32)
        pqb.pq_pack_experts(self.desc, self.A, self.B, self.A8, self.B8, self.hp_scales, self.ws_pack)

    def forward_hp8(self, X=None, Y=None):
        """Forward with the INT8 high-precision branch (after pack() and pack_experts())."""
        pqb.pq_linear_forward_hp8(self.desc, self.X if X is None else X, self.w_s8, self.w_scales, self.A8, self.B8, self.hp_scales,
                                  self.Wr, self.alpha, self.beta, self.Y if Y is None else Y, self.saved, self.ws_fwd)
        return self.Y if Y is None else Y

    def hp8_view(self) -> dict:
        """What forward_hp8 left in the saved h region: codes qh int8 [max_items*128, r] and gamma_h float [max_items*128]."""
        sv = self.saved_view()
        rows = sv["max_items"] * 128
        raw = sv["h"].view(torch.uint8).reshape(-1)
        codes = (rows * self.r + 255) // 256 * 256
        return dict(qh=raw[:rows * self.r].view(torch.int8).view(rows, self.r), gamma_h=raw[codes:codes + 4 * rows].view(torch.float32))

    def backward(self, dY=None):
        pqb.pq_linear_backward(self.desc, self.dY if dY is None else dY, self.X, self.w_s8, self.w_scales, self.A, self.B,
                               self.Wr, self.alpha, self.beta, self.saved, self.dX, self.dW, self.dA, self.dB, self.dWr,
                               self.dalpha, self.dbeta, self.ws_bwd)

    def saved_view(self) -> dict:
        return pqb.pq_saved_view_init(self.desc, self.saved)

    def bwd_view(self) -> dict:
        return pqb.pq_bwd_view_init(self.desc, self.ws_bwd)
