"""Convenience holder for one bound DeTAG state: torch owns the device buffers, the C-ABI library
does every computation.  Used by the tests, the smoke check and the benchmark."""
from __future__ import annotations

from typing import Optional

import numpy as np

from . import binding as B


def _round_up(v: int, m: int) -> int:
    return (v + m - 1) // m * m


class Session:
    """Device buffers x, y, g, a, c ([n][ld] float32) + workspace, bound to a detag_state.

    ``m`` is the matrix a gossip round applies row-wise (an ``inputs.CSR``); ``a``, ``c``, ``x0`` are
    host float32 arrays of shape [n, d] (or None to leave the device buffers uninitialised, e.g.
    when they are filled on the device).  ``external_gradient`` adds the buffer ``g_new`` for
    caller-written gradients and selects that source.
    """

    def __init__(self, m, d: int, K: int, eta: float, alpha: float, a=None, c=None, x0=None, sigma: float = 0.0,
                 seed: int = 0, coord_offset: int = 0, ld: Optional[int] = None, device: str = "cuda:0",
                 observe_gossip: bool = False, variant: int = B.DETAG_VARIANT_AUTO,
                 gradient_point: int = B.DETAG_GRADIENT_AT_NEW_MODEL, algorithm: int = B.DETAG_ALGORITHM_DETAG,
                 external_gradient: bool = False):
        import torch

        if not torch.cuda.is_available():
            raise RuntimeError("the DeTAG step runs on a CUDA device only; none is available")
        self.torch = torch
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.n, self.d = int(m.n), int(d)
        self.ld = _round_up(self.d, 4) if ld is None else int(ld)
        self.state = B.detag_create(self.n, self.d, m.row_ptr, m.col_idx, m.vals, K, eta, alpha)
        shape = (self.n, self.ld)
        self.x = torch.zeros(shape, dtype=torch.float32, device=self.device)
        self.y = torch.zeros(shape, dtype=torch.float32, device=self.device)
        self.g = torch.zeros(shape, dtype=torch.float32, device=self.device)
        self.a = torch.zeros(shape, dtype=torch.float32, device=self.device)
        self.c = torch.zeros(shape, dtype=torch.float32, device=self.device)
        self.y_gossip = torch.zeros(shape, dtype=torch.float32, device=self.device) if observe_gossip else None
        self.workspace = torch.zeros(B.detag_workspace_bytes(self.state) + 256, dtype=torch.uint8, device=self.device)
        pad = (-self.workspace.data_ptr()) % 256
        self._ws_ptr = self.workspace.data_ptr() + pad
        self._ws_bytes = self.workspace.numel() - pad
        for name, host in (("a", a), ("c", c), ("x", x0)):
            if host is not None:
                self.upload(name, host)
        B.detag_bind(self.state, self.ld, self.x, self.y, self.g, self.a, self.c, self._ws_ptr, self._ws_bytes)
        B.detag_set_noise(self.state, sigma, seed, coord_offset)
        if observe_gossip:
            B.detag_observe_gossiped_tracker(self.state, self.y_gossip)
        if variant != B.DETAG_VARIANT_AUTO:
            B.detag_set_variant(self.state, variant)
        if gradient_point != B.DETAG_GRADIENT_AT_NEW_MODEL:
            B.detag_set_gradient_point(self.state, gradient_point)
        if algorithm != B.DETAG_ALGORITHM_DETAG:
            B.detag_set_algorithm(self.state, algorithm)
        # caller-written gradients: the array the caller fills before init and before every step
        self.g_new = torch.zeros(shape, dtype=torch.float32, device=self.device) if external_gradient else None
        if external_gradient:
            B.detag_set_gradient_source(self.state, B.DETAG_GRADIENT_EXTERNAL, self.g_new)

    # ---- data movement (plumbing only)
    def upload(self, name: str, host) -> None:
        t = getattr(self, name)
        src = self.torch.as_tensor(np.ascontiguousarray(host, dtype=np.float32))
        t[:, : self.d].copy_(src)

    def download(self, name: str) -> np.ndarray:
        return getattr(self, name)[:, : self.d].cpu().numpy()

    # ---- the C-ABI calls
    def stream(self):
        return self.torch.cuda.current_stream(self.device)

    def init(self) -> None:
        B.detag_init(self.state, self.stream())

    def step(self, count: int = 1) -> None:
        st = self.stream()
        for _ in range(count):
            B.detag_step(self.state, st)

    def step_many(self, count: int) -> None:
        B.detag_step_many(self.state, count, self.stream())

    def consensus_error(self) -> float:
        return B.detag_consensus_error(self.state, self.stream())

    def status(self) -> None:
        B.detag_status(self.state, self.stream())

    def close(self) -> None:
        if self.state is not None:
            self.torch.cuda.synchronize(self.device)
            B.detag_destroy(self.state)
            self.state = None

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
