"""Backward pass through a stack of linear layers with the chain entry point (vcas_linear_bwd_chain).

Orchestration only: which layer hands what to the next one.  Going down the stack (the order of
backpropagation) every layer receives the list of data the layer above kept - all other data have an
all-zero gradient by then (Sec. 4: the activation gradient gets sparser from layer to layer) - and, when its
incoming gradient is the previous layer's dX, that gradient's row square-norms from the producer's epilogue.
Every step of the method itself runs inside the library's kernels.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

from . import binding as vb


@dataclass
class StackLayer:
    """One linear layer of the stack, in backward order.

    chained: this layer's dY is the dX of the layer before it in backward order.
    H: pre-activation of a GELU feeding THIS layer's input; its dX is multiplied by GELU'(H) (App. E)."""
    name: str
    d_in: int
    d_out: int
    W: torch.Tensor
    X: list            # input activations, one tensor per batch variant [R, d_in]
    dY: list           # incoming gradients per batch variant [R, d_out] (unused when chained)
    H: list | None = None      # pre-activation of the GELU feeding this layer's input, per variant [R, d_in]
    chained: bool = False
    handle: vb.Layer | None = None
    kept: torch.Tensor | None = None
    kept_cnt: torch.Tensor | None = None
    a_out: torch.Tensor | None = None
    dX: torch.Tensor | None = None
    dW: torch.Tensor | None = None


class LinearStack:
    """Owns the per-layer outputs and runs one backward pass per call of `backward`.

    Handles are shared between layers of the same shape (a handle's workspace serves one call at a time and
    the calls of a pass follow one another on one stream)."""

    def __init__(self, layers: list[StackLayer], N: int, T: int, dtype=torch.bfloat16, config=None,
                 gemm_path: int = vb.GEMM_AUTO, skip_dropped_rows: bool = False, overlap_layers: bool = False):
        """skip_dropped_rows: the rows of dX that belong to dropped data are not written (every consumer in the
        stack takes the kept-data list and never reads them); the dX buffers then hold stale rows there."""
        self.layers, self.N, self.T, self.dtype = layers, N, T, dtype
        self.skip_dropped_rows = skip_dropped_rows
        # overlap_layers: a layer's weight-gradient branch is left running while the next layers are scored and
        # their dX products run (vcas_chain_args::defer_join); all handles are joined at the end of the pass
        self.overlap_layers = overlap_layers
        self.R = N * T
        self.handles: dict = {}
        dev = layers[0].W.device
        for i, L in enumerate(layers):
            key = (L.d_in, L.d_out)
            if key not in self.handles:
                self.handles[key] = vb.Layer(N, T, L.d_in, L.d_out, dtype, gemm_path, config)
            L.handle = self.handles[key]
            L.kept = torch.zeros(N, dtype=torch.int32, device=dev)
            L.kept_cnt = torch.zeros(1, dtype=torch.int32, device=dev)
            L.dW = torch.empty(L.d_out, L.d_in, dtype=torch.float32, device=dev)
            nxt = layers[i + 1] if i + 1 < len(layers) else None
            if nxt is not None and nxt.chained:
                assert nxt.d_out == L.d_in, "a chained layer's dY is the previous layer's dX"
                L.dX = torch.empty(self.R, L.d_in, dtype=dtype, device=dev)          # kept: it is the next layer's dY
                L.a_out = torch.empty(self.R, L.handle.chain_parts(), dtype=torch.float32, device=dev)
        # layers whose dX nobody consumes write into one scratch buffer per width
        self._scratch = {}
        for L in layers:
            if L.dX is None:
                if L.d_in not in self._scratch:
                    self._scratch[L.d_in] = torch.empty(self.R, L.d_in, dtype=dtype, device=dev)
                L.dX = self._scratch[L.d_in]

    def backward(self, rho, nu, seed: int, variant: int = 0, hook=None) -> None:
        """One sampled backward pass, top layer first.  rho, nu: per-layer keep ratios in backward order.
        hook(i, layer, after): optional callback before (after=False) and after every layer's call."""
        prev = None
        for i, L in enumerate(self.layers):
            v = variant % len(L.X)
            kw = {}
            if prev is not None:
                kw.update(alive_in=prev.kept, alive_cnt_in=prev.kept_cnt)
            if L.chained:
                dY = prev.dX
                kw.update(a_in=prev.a_out, a_in_parts=prev.handle.chain_parts())
            else:
                dY = L.dY[v]
            H = L.H[v % len(L.H)] if L.H is not None else None
            if hook is not None:
                hook(i, L, False)
            L.handle.linear_bwd_chain(L.X[v], dY, L.W, float(rho[i]), float(nu[i]), seed * len(self.layers) + i,
                                      L.dX, L.dW, H=H, a_out=L.a_out, kept_out=L.kept, kept_cnt_out=L.kept_cnt,
                                      skip_dropped_rows=self.skip_dropped_rows, defer_join=self.overlap_layers, **kw)
            if hook is not None:
                hook(i, L, True)
            prev = L
        if self.overlap_layers:
            for h in self.handles.values():
                h.join()

    def dense_backward(self, variant: int = 0, hook=None) -> None:
        """The exact backward of the same layers (no sampling; the GELU Jacobian where the sampled pass has it):
        the dense comparison."""
        prev = None
        for i, L in enumerate(self.layers):
            v = variant % len(L.X)
            dY = prev.dX if L.chained else L.dY[v]
            if hook is not None:
                hook(i, L, False)
            H = L.H[v % len(L.H)] if L.H is not None else None
            L.handle.dense_bwd(L.X[v], dY, L.W, H=H, dX=L.dX, dW=L.dW)
            if hook is not None:
                hook(i, L, True)
            prev = L

    def probe(self, rho, nu, s: float, seed: int):
        """Alg. 1's probe for every layer (M = number of batch variants).  Returns a [L, 5] device tensor of
        (V_s, V_act, V_w, p_lo, p_hi).  A chained layer is probed on its own gradient variants."""
        dev = self.layers[0].W.device
        out = torch.zeros(len(self.layers), 5, dtype=torch.float32, device=dev)
        for i, L in enumerate(self.layers):
            L.handle.variance_probe(L.X, L.dY, L.W, float(rho[i]), float(nu[i]), float(s), seed + i, out=out[i])
        return out

    def workspace_bytes(self) -> int:
        return sum(h.workspace_bytes() for h in self.handles.values())

    def device_status(self) -> int:
        st = 0
        for h in self.handles.values():
            st = st or h.device_status()
        return st

    def close(self) -> None:
        for h in self.handles.values():
            h.close()
        self.handles = {}
