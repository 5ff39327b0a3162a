"""Sequencing of one outer round on CUDA streams (Algorithm 1's launch / wait structure).

The paper launches Mix1 asynchronously at the top of a round, runs the H inner steps, then
blocks on Mix2, waits for Mix1 and applies the outer optimizer.  On one GPU with K workers as
rows that becomes:

    side stream : Mix1(theta_prev) -> x            (starts once theta_prev is final)
    main stream : inner steps (whatever produces theta_local)
    main stream : wait(Mix1) -> fused outer step (outer grad + Mix2 + Nesterov [+ consensus])

This module only orders C-ABI calls with events; all arithmetic is in the library's kernels.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import (FGD_MIX_IDENTITY, FGD_MIX_MEAN, Context, MixDesc, fgd_consensus_distance, fgd_mix,
               fgd_outer_step_ex)


class OuterRound:
    """Holds the context, the side stream and the Mix1 result buffers for fixed (K, P, ld)."""

    def __init__(self, K: int, P: int, ld: Optional[int] = None, device: int = 0):
        self.ctx = Context(K, P, ld, device)
        self.K, self.P, self.ld = self.ctx.K, self.ctx.P, self.ctx.ld
        self.device = torch.device("cuda", device)
        self.side = torch.cuda.Stream(device=self.device)
        self.cd_sumsq = torch.zeros(K, dtype=torch.float64, device=self.device)
        self._x_vec = None
        self._x_vec2 = None   # second [P] buffer: a step that emits next round's Mix1 writes the one it does not read
        self._x_mat = None
        self._pending = None  # (event, x tensor, x_is_vector)
        self._side_used = False   # has the side stream been given work or a wait (since capture() reset it)?

    # ---- Mix1: non-blocking, on the side stream ------------------------------------------
    def launch_mix1(self, mix1: MixDesc, theta_prev: torch.Tensor) -> None:
        """Start x = Mix1(theta_prev) on the side stream; returns immediately."""
        if mix1.kind == FGD_MIX_IDENTITY:
            raise ValueError("identity Mix1 needs no transfer: pass it as mix1_fused to step()")
        ready = torch.cuda.current_stream(self.device).record_event()
        self.side.wait_event(ready)
        self._side_used = True
        if mix1.kind == FGD_MIX_MEAN:
            if self._x_vec is None:
                self._x_vec = torch.empty(self.P, dtype=torch.float32, device=self.device)
            x, is_vec = self._x_vec, True
        else:
            if self._x_mat is None:
                self._x_mat = torch.empty((self.K, self.ld), dtype=torch.float32, device=self.device)
            x, is_vec = self._x_mat, False
        fgd_mix(self.ctx, mix1, theta_prev, x, out_is_vector=is_vec, stream=self.side)
        self._pending = (self.side.record_event(), x, is_vec)

    # ---- blocking part: wait for Mix1, then the fused outer step ---------------------------
    def step(self, mix2: MixDesc, theta_local, theta_prev, momentum, theta_new, lr: float = 0.7,
             mu: float = 0.9, mix1_fused: Optional[MixDesc] = None, want_cd: bool = True,
             mix2_ranges=None, average_momentum: bool = False, emit_next_mix1: bool = False) -> None:
        """Fused outer step on the current stream.  Uses the pending side-stream Mix1 result,
        or computes Mix1 inside the kernel when ``mix1_fused`` is given.  ``mix2_ranges`` (column
        ranges Mix2 is restricted to) and ``average_momentum`` select the paper's "-subset" and
        GlobalM1S variants.  With ``emit_next_mix1`` (Mix1 = global average) the step also writes
        next round's Mix1 result -- the column mean of theta_new it forms anyway -- and leaves it
        pending, so the next round needs no ``launch_mix1``."""
        cd = self.cd_sumsq if want_cd else None
        x_next = None
        if emit_next_mix1:
            if self._x_vec is None:
                self._x_vec = torch.empty(self.P, dtype=torch.float32, device=self.device)
            if self._x_vec2 is None:
                self._x_vec2 = torch.empty(self.P, dtype=torch.float32, device=self.device)
            reading = self._pending[1] if self._pending is not None else None
            x_next = self._x_vec2 if reading is self._x_vec else self._x_vec
        if mix1_fused is not None:
            fgd_outer_step_ex(self.ctx, mix2, mix1_fused, None, False, theta_local, theta_prev, momentum,
                              theta_new, lr, mu, cd, mix2_ranges, average_momentum, x_next)
            if x_next is not None:
                self._pending = (torch.cuda.current_stream(self.device).record_event(), x_next, True)
            return
        if self._pending is None:
            raise RuntimeError("no Mix1 in flight: call launch_mix1() first or pass mix1_fused")
        ev, x, is_vec = self._pending
        self._pending = None
        torch.cuda.current_stream(self.device).wait_event(ev)
        fgd_outer_step_ex(self.ctx, mix2, None, x, is_vec, theta_local, theta_prev, momentum, theta_new,
                          lr, mu, cd, mix2_ranges, average_momentum, x_next)
        # the side stream may not overwrite x for the next round before this kernel has read it
        done = torch.cuda.current_stream(self.device).record_event()
        self.side.wait_event(done)
        self._side_used = True
        if x_next is not None:
            self._pending = (done, x_next, True)

    # ---- launch-bound sizes: the whole round as one CUDA graph -------------------------------
    def capture(self, body) -> "torch.cuda.CUDAGraph":
        """Capture ``body()`` -- calls of launch_mix1() / step() (and whatever produces theta_local)
        on fixed buffers -- into a CUDA graph and return it; ``replay()`` then runs the round with one
        launch from the host.  The mix descriptors are kernel arguments, so they are frozen into the
        graph: capture one graph per distinct (Mix1, Mix2) pair of a schedule.  Run ``body()`` once
        eagerly beforehand: the first call of a kernel sizes its launch with calls that a capture
        does not allow, and the Mix1 result buffers must exist."""
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self._side_used = False
            body()
            if self._side_used:   # the side stream was pulled into the capture: join it back
                torch.cuda.current_stream(self.device).wait_event(self.side.record_event())
        return g

    def consensus(self, theta) -> torch.Tensor:
        fgd_consensus_distance(self.ctx, theta, self.cd_sumsq)
        return self.cd_sumsq

    def close(self):
        self.ctx.close()
