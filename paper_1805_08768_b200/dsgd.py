"""Algorithm 1 end to end on one GPU: synchronous distributed SGD with communication delay.

Every client i of a round (Algorithm 1, client lines) starts from the common weights W, runs
``delay`` local SGD iterations on its own data (``SGD_n`` -- Section 2, "Communication Delay":
the weight update is sent only every n-th iteration), adds what it did not get to send in earlier
rounds, compresses, keeps the remainder and encodes:

    dW_i  <-  R_i + (SGD_n(W, D_i) - W)
    dW_i* <-  compress(dW_i),   R_i <- dW_i - dW_i*,   msg_i <- encode(dW_i*)

and the server (or, here, every holder of the weights) decodes and averages:

    W  <-  W + 1/M * sum_i decode(msg_i)

The clients are simulated as buffers on one GPU.  This module only moves arguments: the
compression, the coding and the decode-and-apply are the CUDA library's calls
(``sbc_encode_batch`` over a client's tensors, ``sbc_decode_apply`` over the M messages of a
tensor); the local SGD iterations are the caller's (a callback), since they belong to the model and
not to the method.  ``ToyRegression`` is a small seeded stand-in for such a model.
"""
from __future__ import annotations

from typing import Callable, List, Optional, Sequence

import torch

from . import binding


class DelayedSGD:
    """M simulated clients sharing one replica of the weights.

    ``weights``: list of float32 CUDA tensors (updated in place by every round).
    ``local_update(client, weights, delay) -> list of tensors``: runs ``delay`` SGD iterations for
    that client starting from ``weights`` (without changing them) and returns W_after - W per tensor.
    ``momenta``: optional per-tensor momentum buffers of the caller's optimiser; zeroed at every
    transmitted position (momentum masking, Supplement)."""

    def __init__(self, weights: Sequence[torch.Tensor], n_clients: int, p: float, delay: int,
                 local_update: Callable[[int, Sequence[torch.Tensor], int], List[torch.Tensor]],
                 momenta: Optional[Sequence[torch.Tensor]] = None):
        if n_clients < 1 or delay < 1:
            raise ValueError("need at least one client and a delay of at least one iteration")
        self.weights = list(weights)
        self.flat = [w.view(-1) for w in self.weights]
        self.n_clients, self.p, self.delay = n_clients, float(p), int(delay)
        self.local_update = local_update
        self.momenta = [m.view(-1) for m in momenta] if momenta is not None else None
        dev = self.weights[0].device
        sizes = [w.numel() for w in self.weights]
        self.sizes = sizes
        ps = [self.p] * len(sizes)
        self.ps = ps
        self.residuals = [[torch.zeros(n, dtype=torch.float32, device=dev) for n in sizes] for _ in range(n_clients)]
        self.capacity = [binding.sbc_stream_bytes(n, self.p) for n in sizes]
        self.messages = [[torch.zeros(c, dtype=torch.uint8, device=dev) for c in self.capacity] for _ in range(n_clients)]
        self.mus = [[torch.zeros(1, dtype=torch.float32, device=dev) for _ in sizes] for _ in range(n_clients)]
        self.workspace = torch.empty(binding.sbc_workspace_bytes_batch(sizes, ps), dtype=torch.uint8, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.rounds_done = 0
        self.last_updates: List[List[torch.Tensor]] = []   # the clients' local updates of the last round (for inspection)

    def round(self) -> None:
        """One communication round of Algorithm 1 for all clients."""
        self.last_updates = []
        for c in range(self.n_clients):
            upd = [u.contiguous().view(-1) for u in self.local_update(c, self.weights, self.delay)]
            self.last_updates.append(upd)
            binding.sbc_encode_batch(upd, self.residuals[c], self.ps, self.messages[c], self.mus[c], self.workspace)
        scale = 1.0 / self.n_clients
        for t in range(len(self.sizes)):
            binding.sbc_decode_apply([self.messages[c][t] for c in range(self.n_clients)], scale, self.flat[t],
                                     self.momenta[t] if self.momenta is not None else None, self.status,
                                     sizes=[self.capacity[t]] * self.n_clients)
        self.rounds_done += 1

    def check(self) -> None:
        """Synchronise and raise if a decode reported a damaged message."""
        torch.cuda.synchronize()
        if int(self.status.item()) != 0:
            raise RuntimeError(f"decode status {int(self.status.item())}")


class ToyRegression:
    """A two-layer perceptron on seeded synthetic regression data, one shard per client; plain SGD.
    Stands in for the paper's networks and data sets, none of which are used here."""

    def __init__(self, n_clients: int, device: torch.device, in_dim: int = 64, hidden: int = 256, out_dim: int = 8,
                 samples_per_client: int = 512, batch: int = 64, lr: float = 0.05, seed: int = 0):
        g = torch.Generator(device="cpu").manual_seed(seed)
        teacher = torch.randn(in_dim, out_dim, generator=g) / in_dim ** 0.5
        self.x = [torch.randn(samples_per_client, in_dim, generator=g).to(device) for _ in range(n_clients)]
        self.y = [(torch.tanh(x.cpu() @ teacher) + 0.01 * torch.randn(samples_per_client, out_dim, generator=g)).to(device)
                  for x in self.x]
        self.weights = [(torch.randn(in_dim, hidden, generator=g) / in_dim ** 0.5).to(device),
                        torch.zeros(hidden, device=device),
                        (torch.randn(hidden, out_dim, generator=g) / hidden ** 0.5).to(device),
                        torch.zeros(out_dim, device=device)]
        self.batch, self.lr = batch, lr
        self.cursor = [0] * n_clients

    @staticmethod
    def _forward(params, x):
        w1, b1, w2, b2 = params
        return torch.tanh(x @ w1 + b1) @ w2 + b2

    def loss(self, params=None) -> float:
        params = self.weights if params is None else params
        with torch.no_grad():
            return float(sum(torch.mean((self._forward(params, x) - y) ** 2) for x, y in zip(self.x, self.y)) / len(self.x))

    def local_update(self, client: int, weights: Sequence[torch.Tensor], delay: int) -> List[torch.Tensor]:
        """``delay`` SGD iterations on the client's shard, starting from ``weights``; returns W_after - W."""
        params = [w.detach().clone().requires_grad_(True) for w in weights]
        x, y = self.x[client], self.y[client]
        for _ in range(delay):
            lo = self.cursor[client]
            self.cursor[client] = (lo + self.batch) % (x.shape[0] - self.batch + 1)
            loss = torch.mean((self._forward(params, x[lo:lo + self.batch]) - y[lo:lo + self.batch]) ** 2)
            grads = torch.autograd.grad(loss, params)
            with torch.no_grad():
                for w, gr in zip(params, grads):
                    w -= self.lr * gr
        return [(w.detach() - w0).contiguous() for w, w0 in zip(params, weights)]
