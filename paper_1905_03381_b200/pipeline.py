"""Assistant and Boss as two CUDA streams with a bounded queue of screened batches between them
(Sec. "Asynchronous joint learning with CPU/GPU"; Algorithms 2 and 3: the Assistant thread fills the Boss queue up to k batches and otherwise
trains on the (batch, losses) items the Boss hands back).

The paper runs the two workers as threads that meet in two queues.  On one GPU the same schedule is
stream order: every call of the library only enqueues work, so the host loop below fixes one order
of events and CUDA events carry the two queue hand-offs.

  Assistant stream : screen pool j (score -> shrink -> ordered batch list) whenever the Boss queue
                     holds fewer than `depth` batches beyond the one the Boss needs next, else one
                     update on the oldest (batch, losses) item.
  Boss stream      : per-instance losses of batch t (the caller's `boss` function; a real Boss also
                     runs its own forward/backward there), after the event that says batch t is
                     screened; its own event releases the Assistant's update.

Batch j is therefore screened with the parameters after max(0, j - depth) updates; depth = 0 is the
sequential path.  The screened batches live in a ring of depth + 1 slots (index list, device count,
losses); nothing crosses to the host.  Host logic only: every step of the data path is a call into
the CUDA library.
"""
from __future__ import annotations

from typing import Callable, Optional

import torch

from . import binding as B


class StreamPipeline:
    """Two library contexts (one per stream) and the ring of screened batches between them."""

    def __init__(self, depth: int, max_rows: int, max_d: int, capacity: int, max_hidden: int = 0, device="cuda:0",
                 slots: Optional[int] = None, boss_max_rows: Optional[int] = None):
        if depth < 0:
            raise ValueError("depth must be >= 0")
        self.depth = depth
        self.slots = max(depth + 1, slots or 0)
        self.capacity = capacity
        self.device = torch.device(device)
        with torch.cuda.device(self.device):
            self.assistant_stream = torch.cuda.Stream(self.device)
            self.boss_stream = torch.cuda.Stream(self.device)
            self.assistant_ctx = B.AutoAssist(max_rows, max_d, max_hidden, device=self.device, stream=self.assistant_stream)
            self.boss_ctx = B.AutoAssist(boss_max_rows or max(capacity, 1), 16, 0, device=self.device, stream=self.boss_stream)
            self.idx = torch.zeros((self.slots, max(capacity, 1)), dtype=torch.int32, device=self.device)
            self.count = torch.zeros((self.slots, 1), dtype=torch.int32, device=self.device)
            self.loss = torch.zeros((self.slots, max(capacity, 1)), dtype=torch.float32, device=self.device)
            self._screened = [torch.cuda.Event() for _ in range(self.slots)]
            self._lossed = [torch.cuda.Event() for _ in range(self.slots)]

    def close(self):
        self.assistant_ctx.close()
        self.boss_ctx.close()

    def launch_count(self) -> int:
        return self.assistant_ctx.aa_launch_count() + self.boss_ctx.aa_launch_count()

    def device_status(self) -> int:
        a = self.assistant_ctx.aa_device_status()
        b = self.boss_ctx.aa_device_status()
        return a if a != B.AA_OK else b

    def run(self, n_steps: int, features: Callable, boss: Callable, assistant: B.aa_assistant, mix: float, seed: int,
            lr: float, threshold=None, first_step: int = 0, adam: Optional[B.aa_adam] = None,
            after_update: Optional[Callable] = None):
        """Enqueue n_steps of the schedule and return without synchronising.

        features(j, row_idx) -> aa_feat of pool j (row_idx None: the whole pool as candidates; else the batch rows
            selected by that device index list, n_rows = its length).
        boss(t, ctx, idx, count_dev, out_loss): enqueue, on the Boss stream (current while it is called) and through
            the Boss context `ctx`, the losses of batch t: out_loss[i] for the instance idx[i], i < count_dev[0].
        after_update(t): optional, called with the Assistant stream current right after update t is enqueued.
        Pool j is screened with Philox step first_step + j.  The caller's current stream is ordered before the first
        and after the last piece of work.
        """
        A, Bs = self.assistant_stream, self.boss_stream
        cur = torch.cuda.current_stream(self.device)
        A.wait_stream(cur)
        Bs.wait_stream(cur)
        actx = self.assistant_ctx
        next_screen = 0
        for t in range(n_steps):
            # Assistant: sampling comes before updating while the Boss queue is short (Algorithm 2)
            while next_screen < n_steps and next_screen <= t + self.depth:
                j, s = next_screen, next_screen % self.slots
                actx.aa_score_shrink(features(j, None), assistant, mix, seed, first_step + j, self.idx[s], self.count[s])
                self._screened[s].record(A)
                next_screen += 1
            s = t % self.slots
            # Boss: pop batch t, losses, push (batch, losses) (Algorithm 3)
            Bs.wait_event(self._screened[s])
            with torch.cuda.stream(Bs):
                boss(t, self.boss_ctx, self.idx[s], self.count[s], self.loss[s])
            self._lossed[s].record(Bs)
            # Assistant: pop that item, gradient, update
            A.wait_event(self._lossed[s])
            batch = features(t, self.idx[s])
            if adam is None:
                actx.aa_assistant_step(batch, self.loss[s], assistant, lr, threshold=threshold, count_dev=self.count[s])
            else:
                actx.aa_assistant_step_adam(batch, self.loss[s], assistant, adam, lr, threshold=threshold,
                                            count_dev=self.count[s])
            if after_update is not None:
                with torch.cuda.stream(A):
                    after_update(t)
        cur.wait_stream(A)
        cur.wait_stream(Bs)
