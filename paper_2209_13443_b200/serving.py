"""Host-side serving loops over the C-ABI library.

``FluidServer.serve`` is the paper's exit-aware preemptive scheduler (Algorithm 1) with its SLO-aware preemption
criterion (Eq. 3-4): the active batch runs one subnet at a time; behind every exit the scheduler learns B_exit, and
while the batch has room and the queue is not empty it parks the remaining samples where they are (activations
already live in device memory: Section III-B, Overhead), lets newly queued requests catch up to the same exit and
merges the two.  Backfilling is per exit and non-recursive.  A backfill is taken only if the predicted extra time,
T_{0:i} at the size of the new batch plus T_{i+1:L-1} at the merged size, is below the slack T_SLO minus the time
the oldest sample of the active batch has spent so far; the exit-level latencies come from an N_exits x B_max table
measured on the device (Section III-B, Exit-Level Latency Prediction).  With T_SLO = infinity every backfill that
fits is taken.

Two comparison policies of the paper's evaluation run on the same calls: ``serve_serial`` (one request at a time,
Section IV "SERIAL") and ``serve_adaptive_batching`` (the <B_max, T_timeout> policy of Section II-A: a batch is
issued when B_max requests wait or the oldest has waited T_timeout, and then runs through its exits with no refill).

All device work goes through ee_stage_run / ee_batch_refill / ee_gather_survivors; this file keeps the queue, the
clocks and the bookkeeping.  The building blocks are the library's own operations: admit (queue), form_batch (gather
of the requests' inputs), run_stage (one subnet + exit), catch_up (a new batch up to an exit), merge (refill).
"""
from __future__ import annotations

import time
from collections import deque
from typing import Callable, Optional, Sequence

import numpy as np
import torch

from . import binding as eb


class _Clock:
    """Virtual (advanced by a stage-time model) or wall clock."""

    def __init__(self, stage_time):
        self.stage_time = stage_time
        self.t0 = time.perf_counter()
        self.t = 0.0

    @property
    def virtual(self):
        return self.stage_time is not None

    def now(self):
        if not self.virtual:
            self.t = time.perf_counter() - self.t0
        return self.t

    def after_stage(self, s, n):
        if self.virtual:
            self.t += self.stage_time(s, n)
        return self.now()

    def wait_until(self, when):
        if self.virtual:
            self.t = max(self.t, float(when))
        else:
            while time.perf_counter() - self.t0 < when:
                pass
        return self.now()


class FluidServer:
    def __init__(self, spec, model: Optional[eb.EEModel] = None):
        self.spec = spec
        self.m = model or eb.EEModel(spec)
        self.n_stages = self.m.n_stages
        self.bmax = spec.max_batch
        # two buffer sets: the active batch and the batch that catches up to it
        self.act = [eb.StageBuffers(self.m, s, with_logits=False) for s in range(self.n_stages)]
        self.new = [eb.StageBuffers(self.m, s, with_logits=False) for s in range(self.n_stages)]
        self.ws = self.m.workspace()
        td = eb.torch_dtype(spec.dtype)
        shape = (self.bmax, spec.in_h, spec.in_w, spec.in_c)
        self.in_act = torch.empty(shape, dtype=td, device="cuda")
        self.in_new = torch.empty(shape, dtype=td, device="cuda")
        self.ids_act = torch.empty(self.bmax, dtype=torch.int32, device="cuda")
        self.ids_new = torch.empty(self.bmax, dtype=torch.int32, device="cuda")
        self.idx_dev = torch.empty(self.bmax, dtype=torch.int32, device="cuda")
        self.cnt_dev = torch.empty(1, dtype=torch.int32, device="cuda")
        # pinned staging: request rows / ids / count on their way in, exit masks and classes on their way out
        self.h_idx = torch.empty(self.bmax, dtype=torch.int32).pin_memory()
        self.h_ids = torch.empty(self.bmax, dtype=torch.int32).pin_memory()
        self.h_cnt = torch.empty(1, dtype=torch.int32).pin_memory()
        self.h_mask = torch.empty(self.bmax, dtype=torch.uint8).pin_memory()
        self.h_pred = torch.empty(self.bmax, dtype=torch.int32).pin_memory()
        self.stage_in_bytes = [self.m.query(s)["in_bytes_per_sample"] for s in range(self.n_stages)]

    # ------------------------------------------------------------------ measured exit-level latency table

    def measure_latency_table(self, reps: int = 5) -> np.ndarray:
        """The N_exits x B_max look-up table of the scheduler: seconds one ee_stage_run of subnet s takes at batch
        b (CUDA events around ``reps`` replays on random features; column b - 1 holds batch b)."""
        lut = np.zeros((self.n_stages, self.bmax))
        td = eb.torch_dtype(self.spec.dtype)
        a, b_ev = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for s in range(self.n_stages):
            qi = self.m.query(s)
            x = (torch.randn(self.bmax, qi["in_h"], qi["in_w"], qi["in_c"], device="cuda") * 0.5).to(td)
            for b in range(1, self.bmax + 1):
                self.m.stage_run(s, x, b, self.new[s], self.ws, self.ids_new)        # first call: plain launches / capture
                a.record()
                for _ in range(reps):
                    self.m.stage_run(s, x, b, self.new[s], self.ws, self.ids_new)
                b_ev.record()
                b_ev.synchronize()
                lut[s, b - 1] = a.elapsed_time(b_ev) * 1e-3 / reps
        return lut

    # ------------------------------------------------------------------ building blocks

    def form_batch(self, pool, rows: Sequence[int], req_ids: Sequence[int], feat, ids):
        """Gathers the requests' inputs (rows of ``pool``) to the front of the batch buffer ``feat``: one small pinned
        upload of the row list, the ids and the count, then one ee_gather_survivors."""
        n = len(rows)
        self.h_idx[:n] = torch.as_tensor(np.asarray(rows, dtype=np.int32))
        self.h_ids[:n] = torch.as_tensor(np.asarray(req_ids, dtype=np.int32))
        self.h_cnt[0] = n
        self.idx_dev[:n].copy_(self.h_idx[:n], non_blocking=True)
        ids[:n].copy_(self.h_ids[:n], non_blocking=True)
        self.cnt_dev.copy_(self.h_cnt, non_blocking=True)
        eb.gather_survivors(pool, self.stage_in_bytes[0], self.idx_dev, self.cnt_dev, n, feat)

    def run_stage(self, s, feat, ids_dev, members, bufs, clock: _Clock, out):
        """One subnet and its exit on the batch ``members`` (request numbers, in batch order).  The exit mask and the
        classes travel to pinned host memory behind the stage; the host waits for them once.  Records the requests
        that leave; returns those that stay."""
        n = len(members)
        self.m.stage_run(s, feat, n, bufs[s], self.ws, ids_dev)
        self.h_mask[:n].copy_(bufs[s].exit_mask[:n], non_blocking=True)
        self.h_pred[:n].copy_(bufs[s].pred[:n], non_blocking=True)
        torch.cuda.current_stream().synchronize()            # B_exit (and who left) reaches the scheduler
        now = clock.after_stage(s, n)
        out["launches"].append((s, tuple(members)))
        mask, pred = self.h_mask[:n].numpy(), self.h_pred[:n].numpy()
        stay = []
        for j, r in enumerate(members):
            if mask[j]:
                out["finish"][r] = now
                out["exit_stage"][r] = s
                out["pred"][r] = int(pred[j])
            else:
                stay.append(r)
        assert len(stay) == int(bufs[s].n_surv_host[0])
        return stay

    def catch_up(self, pool, image_of, members, upto, clock, out):
        """A newly issued batch runs from the input to exit ``upto``.  Returns (survivors, their features, their ids)."""
        self.form_batch(pool, [image_of[r] for r in members], members, self.in_new, self.ids_new)
        feat, ids = self.in_new, self.ids_new
        for j in range(upto + 1):
            members = self.run_stage(j, feat, ids, members, self.new, clock, out)
            feat, ids = self.new[j].features_out, self.new[j].ids_out
            if not members:
                break
        return members, feat, ids

    def merge(self, boundary, feat, ids, members, new_feat, new_ids, new_members):
        """ee_batch_refill: the caught-up samples are appended behind the parked ones."""
        n_acc, n_mer = self.m.batch_refill(boundary, feat, ids, len(members), new_feat, new_ids, len(new_members))
        assert n_acc == len(new_members) and n_mer == len(members) + len(new_members)
        return members + new_members

    @staticmethod
    def _result(n):
        return {"finish": np.zeros(n), "exit_stage": np.full(n, -1), "pred": np.full(n, -1), "launches": [],
                "preemptions": 0, "declined": 0}

    # ------------------------------------------------------------------ Algorithm 1

    def serve(self, arrivals: np.ndarray, image_of: Sequence[int], pool: torch.Tensor,
              stage_time: Optional[Callable[[int, int], float]] = None, slo: float = float("inf"),
              latency: Optional[Callable[[int, int], float]] = None):
        """Serves requests r = 0..n-1 arriving at ``arrivals[r]`` (sorted, seconds) and carrying image
        ``pool[image_of[r]]``.  With ``stage_time(stage, batch)`` the clock is virtual (deterministic batch
        compositions); without it the wall clock is used and the loop waits for arrivals.
        ``slo`` is T_SLO in seconds; ``latency(stage, batch)`` is the exit-level latency table the preemption
        criterion consults (default: ``stage_time``; required on the wall clock when ``slo`` is finite).
        Returns dict(finish, exit_stage, pred, launches, preemptions, declined)."""
        n = len(arrivals)
        out = self._result(n)
        latency = latency or stage_time
        if np.isfinite(slo) and latency is None:
            raise ValueError("a finite SLO needs the exit-level latency table (latency=...)")
        clock = _Clock(stage_time)
        queue: deque = deque()
        state = {"next": 0}

        def admit():
            now = clock.now()
            while state["next"] < n and arrivals[state["next"]] <= now:
                queue.append(state["next"])
                state["next"] += 1

        def predicted(first, last, batch):
            return sum(latency(j, batch) for j in range(first, last + 1))

        def may_preempt(members, exit_idx, n_new):
            """The SLO-aware criterion: the backfill must not push the oldest active sample past its SLO."""
            if not members or not np.isfinite(slo):
                return True
            slack = slo - (clock.now() - min(arrivals[r] for r in members))
            overhead = predicted(0, exit_idx, n_new) + predicted(exit_idx + 1, self.n_stages - 1, len(members) + n_new)
            return overhead < slack

        while state["next"] < n or queue:
            admit()
            if not queue:
                clock.wait_until(arrivals[state["next"]])
                admit()
            members = [queue.popleft() for _ in range(min(len(queue), self.bmax))]
            self.form_batch(pool, [image_of[r] for r in members], members, self.in_act, self.ids_act)
            feat, ids = self.in_act, self.ids_act
            for exit_idx in range(self.n_stages - 1):       # every exit but the last is a preemption point
                members = self.run_stage(exit_idx, feat, ids, members, self.act, clock, out)
                feat, ids = self.act[exit_idx].features_out, self.act[exit_idx].ids_out     # parked at the boundary
                while len(members) < self.bmax:
                    admit()
                    n_new = min(len(queue), self.bmax - len(members))
                    if n_new == 0:
                        break
                    if not may_preempt(members, exit_idx, n_new):
                        out["declined"] += 1
                        break
                    out["preemptions"] += 1
                    fresh = [queue.popleft() for _ in range(n_new)]
                    fresh, f_feat, f_ids = self.catch_up(pool, image_of, fresh, exit_idx, clock, out)
                    if fresh:
                        members = self.merge(exit_idx + 1, feat, ids, members, f_feat, f_ids, fresh)
                if not members:
                    break
            if members:
                members = self.run_stage(self.n_stages - 1, feat, ids, members, self.act, clock, out)
                assert not members
        torch.cuda.synchronize()
        return out

    # ------------------------------------------------------------------ comparison policies

    def _run_to_completion(self, pool, image_of, members, clock, out):
        self.form_batch(pool, [image_of[r] for r in members], members, self.in_act, self.ids_act)
        feat, ids = self.in_act, self.ids_act
        for s in range(self.n_stages):
            members = self.run_stage(s, feat, ids, members, self.act, clock, out)
            if not members:
                break
            feat, ids = self.act[s].features_out, self.act[s].ids_out

    def serve_serial(self, arrivals, image_of, pool, stage_time=None):
        """One request at a time in arrival order, each through its exits alone."""
        return self.serve_adaptive_batching(arrivals, image_of, pool, max_batch=1, timeout=0.0, stage_time=stage_time)

    def serve_adaptive_batching(self, arrivals, image_of, pool, max_batch: Optional[int] = None, timeout: float = 0.0,
                                stage_time=None):
        """The <B_max, T_timeout> policy: a batch is issued as soon as ``max_batch`` requests wait or the oldest
        waiting request has waited ``timeout`` seconds; it then runs through all its exits (shrinking, never refilled)."""
        n = len(arrivals)
        out = self._result(n)
        bmax = min(max_batch or self.bmax, self.bmax)
        clock = _Clock(stage_time)
        queue: deque = deque()
        nxt = 0
        while nxt < n or queue:
            now = clock.now()
            while nxt < n and arrivals[nxt] <= now:
                queue.append(nxt)
                nxt += 1
            if not queue:
                clock.wait_until(arrivals[nxt])
                continue
            deadline = arrivals[queue[0]] + timeout
            if len(queue) < bmax and now < deadline and nxt < n:
                clock.wait_until(min(deadline, arrivals[nxt]))     # the next event: a new arrival or the time-out
                continue
            members = [queue.popleft() for _ in range(min(len(queue), bmax))]
            self._run_to_completion(pool, image_of, members, clock, out)
        torch.cuda.synchronize()
        return out
