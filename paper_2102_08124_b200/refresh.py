"""Periodic mask refresh for sparse training from scratch (Section 4.1 of the paper): the optimizer keeps
updating dense copies of the weights, forward and backward use the masked weights, and every `period`
iterations (40 in the paper) the transposable masks of all layers are re-derived by one batched call.

Everything the refresh does on the GPU runs in this library's kernels (the prepared batched search and the
count of changed mask bits), recorded once into a CUDA graph and replayed; torch only provides the tensors,
the stream and the graph object."""
from __future__ import annotations

from typing import List, Sequence

from . import binding as tm


class MaskRefresher:
    """masks / masked_weights are refreshed in place; `changed_bits` records, per refresh, how many mask bits flipped."""

    def __init__(self, weights: Sequence, N: int = 4, M: int = 8, period: int = 40, method: int = tm.TM_APPROX, use_graph: bool = True):
        import torch
        self.weights = list(weights)
        self.N, self.M, self.period, self.method = N, M, period, method
        dev = self.weights[0].device
        words = [W.shape[0] * tm.tm_mask_words_per_row(W.shape[1]) for W in self.weights]
        self._flat = torch.zeros((sum(words),), dtype=torch.int32, device=dev)       # all masks, one buffer
        self._prev = torch.zeros_like(self._flat)
        self.masks, off = [], 0
        for W, n in zip(self.weights, words):
            self.masks.append(self._flat[off:off + n].view(W.shape[0], -1)); off += n
        self.plan = tm.tm_plan_create(self.weights, N, M, method, masks=self.masks)
        self.masked_weights = self.plan.batch.maskeds
        self.objectives, self.status = self.plan.batch.objectives, self.plan.batch.status
        self._distance = torch.zeros((1,), dtype=torch.int64, device=dev)
        self._aux_ws = torch.empty((tm.tm_aux_workspace_bytes(),), dtype=torch.uint8, device=dev)
        self.changed_bits: List[int] = []
        self.refreshes = 0
        self._graph = None
        self._refresh_eager()                                   # first masks; also warms every kernel up before a capture
        self.changed_bits.clear(); self.refreshes = 0
        if use_graph:
            torch.cuda.synchronize(dev)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                self._enqueue()
            self._graph = g

    def _enqueue(self):
        self._prev.copy_(self._flat)
        tm.tm_plan_run(self.plan)
        tm.tm_mask_hamming(self._flat, self._prev, distance_out=self._distance, workspace=self._aux_ws)

    def _refresh_eager(self):
        self._enqueue()
        self.changed_bits.append(int(self._distance.item()))
        self.refreshes += 1

    def refresh(self):
        """Re-derives every mask from the current dense weights; returns the number of mask bits that changed."""
        if self._graph is None:
            self._refresh_eager()
        else:
            self._graph.replay()
            self.changed_bits.append(int(self._distance.item()))
            self.refreshes += 1
        return self.changed_bits[-1]

    def step(self, iteration: int) -> bool:
        """Call once per training iteration (after the optimizer step); refreshes when iteration % period == 0."""
        if iteration % self.period == 0:
            self.refresh()
            return True
        return False


def masked_linear(x, weight_dense, weight_masked):
    """y = x @ (W*S)^T with the straight-through treatment of the dense copy: the forward product and the
    input gradient use the masked weights (both are N:M-sparse products thanks to the transposable mask, Eq. bwd
    of the paper's introduction), the weight gradient goes to the dense copy unmasked."""
    import torch

    class _Fn(torch.autograd.Function):
        @staticmethod
        def forward(ctx, x_, wd, wm):
            ctx.save_for_backward(x_, wm)
            return x_ @ wm.t()

        @staticmethod
        def backward(ctx, gy):
            x_, wm = ctx.saved_tensors
            gx = gy @ wm                                         # dL/dX = (W*S)^T-product: the transposed operand is N:M sparse too
            gw = gy.reshape(-1, gy.shape[-1]).t() @ x_.reshape(-1, x_.shape[-1])
            return gx, gw, None

    return _Fn.apply(x, weight_dense, weight_masked)
