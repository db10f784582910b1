"""A pipeline-stage boundary over torch.distributed (Algorithm 1, lines 4-7).

Forward: the sending stage encodes its output activations with the TAH-Quant codec and sends the packed
bytes; the receiving stage decodes them.  Backward: the receiving stage sends the gradient with respect to
those activations through the fixed-point compressor (pre-scaled, g_hat = Q(c g) / c), the sending stage
decodes it.  The packed buffers have a size that depends on the parameters only, so both sides allocate
once and the transport sees fixed-shape byte tensors (Sec. 3.4).

The codec runs on each rank's own GPU and stream; the only inter-GPU step is the point-to-point transfer
of the packed buffer (NCCL send/recv over NVLink when the process group is NCCL).  `codec` is injectable so
that the transport can be exercised without a GPU.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable, Protocol

import torch
import torch.distributed as dist


class Codec(Protocol):
    """encode(x) -> uint8 tensor of fixed size; decode(bytes) -> tensor."""

    nbytes: int

    def encode(self, x: torch.Tensor) -> torch.Tensor: ...

    def decode(self, packed: torch.Tensor) -> torch.Tensor: ...


class TahqCodec:
    """Forward codec: tahq_encode / tahq_decode with a workspace and a packed buffer allocated once."""

    def __init__(self, tokens: int, hidden: int, dtype: torch.dtype, device, **params):
        from . import binding as T
        self.T = T
        self.p = T.Params(tokens=tokens, hidden=hidden, dtype={torch.float32: T.F32, torch.bfloat16: T.BF16}[dtype],
                          **params)
        self.nbytes = T.packed_bound(self.p)
        self.ws = T.alloc_workspace(self.p, device)
        self.packed = T.alloc_packed(self.p, device)
        self.out = torch.empty((tokens, hidden), dtype=dtype, device=device)

    def encode(self, x):
        return self.T.encode(self.p, x, packed=self.packed, ws=self.ws)

    def decode(self, packed):
        return self.T.decode(self.p, packed, out=self.out, ws=self.ws)


class QNaiveCodec:
    """Backward codec: tahq_qnaive_encode / tahq_qnaive_decode."""

    def __init__(self, tokens: int, hidden: int, dtype: torch.dtype, device, bits: int = 6, prescale: float = 1.0,
                 per_tensor: int = 0):
        from . import binding as T
        self.T = T
        self.p = T.QNaiveParams(tokens=tokens, hidden=hidden,
                                dtype={torch.float32: T.F32, torch.bfloat16: T.BF16}[dtype], bits=bits,
                                per_tensor=per_tensor, prescale=prescale)
        self.nbytes = T.qnaive_packed_bound(self.p)
        self.ws = torch.empty(T.qnaive_workspace_bound(self.p), dtype=torch.uint8, device=device)
        self.packed = torch.empty(self.nbytes, dtype=torch.uint8, device=device)
        self.out = torch.empty((tokens, hidden), dtype=dtype, device=device)

    def encode(self, x):
        return self.T.qnaive_encode(self.p, x, packed=self.packed, ws=self.ws)[0]

    def decode(self, packed):
        return self.T.qnaive_decode(self.p, packed, out=self.out, ws=self.ws)[0]


@dataclass
class Boundary:
    """One boundary between stage `lower` (rank that produces activations) and stage `upper`."""

    lower: int
    upper: int
    forward: Codec
    backward: Codec
    recv_buffer: Callable[[int], torch.Tensor]   # nbytes -> uint8 tensor on this rank's device

    def send_activations(self, x: torch.Tensor) -> None:          # on `lower` (Algorithm 1 line 4)
        dist.send(self.forward.encode(x), dst=self.upper)

    def recv_activations(self) -> torch.Tensor:                    # on `upper` (line 5)
        buf = self.recv_buffer(self.forward.nbytes)
        dist.recv(buf, src=self.lower)
        return self.forward.decode(buf)

    def send_gradient(self, g: torch.Tensor) -> None:              # on `upper` (line 6)
        dist.send(self.backward.encode(g), dst=self.lower)

    def recv_gradient(self) -> torch.Tensor:                       # on `lower` (line 7)
        buf = self.recv_buffer(self.backward.nbytes)
        dist.recv(buf, src=self.upper)
        return self.backward.decode(buf)
