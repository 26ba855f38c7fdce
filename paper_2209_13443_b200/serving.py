"""Host-side serving loop over the C-ABI library: the exit-aware preemptive scheduling method
(Algorithm 1) with its SLO-aware preemption criterion (Eq. 3-4).

At every exit the scheduler learns B_exit, and while the batch has room and the queue is not
empty it preempts the active batch (which simply stays parked in its HBM buffer: activations are
already in device memory, Section III-B "Overhead"), lets B_incr = min(N_Q, B_max - B_rem) new
requests catch up to the same exit, and merges them (B_merged = B_rem + B_incr - B_exit).
Backfilling is per exit and non-recursive.  A backfill is taken only if it cannot push the oldest
sample of the active batch past the latency SLO: T_overhead = T_{0:i}(B_incr) + T_{i+1:L-1}(B_merged)
must be below T_slack = T_SLO - (T_wait + T_exec so far).  The exit-level latencies come from a
N_exits x B_max table measured on the device (``measure_latency_table``; Section III-B, Exit-Level
Latency Prediction).  With T_SLO = infinity every backfill that fits is taken.

All device work goes through ``ee_stage_run`` / ``ee_batch_refill`` / ``ee_gather_survivors``;
this file only keeps the queue, the clocks and the bookkeeping.
"""
from __future__ import annotations

import time
from collections import deque
from typing import Callable, Optional, Sequence

import numpy as np
import torch

from . import binding as eb


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
        self.stage_in_bytes = [self.m.query(s)["in_bytes_per_sample"] for s in range(self.n_stages)]

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

    def _form_batch(self, pool, rows: Sequence[int], req_ids: Sequence[int], feat, ids):
        """Copies the requested pool images into the front of ``feat`` (the batch buffer)."""
        n = len(rows)
        self.idx_dev[:n] = torch.as_tensor(np.asarray(rows, dtype=np.int32), device="cuda")
        ids[:n] = torch.as_tensor(np.asarray(req_ids, dtype=np.int32), device="cuda")
        self.cnt_dev.fill_(n)
        eb.gather_survivors(pool, self.stage_in_bytes[0], self.idx_dev, self.cnt_dev, n, feat)

    def _run(self, s, feat, ids_dev, ids_host, bufs, now, clock, stage_time, out):
        """One ee_stage_run; records the requests that leave.  Returns (survivor ids, new time)."""
        n = len(ids_host)
        self.m.stage_run(s, feat, n, bufs[s], self.ws, ids_dev)
        torch.cuda.current_stream().synchronize()            # B_exit reaches the scheduler
        mask = bufs[s].exit_mask[:n].cpu().numpy()
        pred = bufs[s].pred[:n].cpu().numpy()
        now = clock() if stage_time is None else now + stage_time(s, n)
        out["launches"].append((s, tuple(ids_host)))
        rem = []
        for j, r in enumerate(ids_host):
            if mask[j]:
                out["finish"][r] = now
                out["exit_stage"][r] = s
                out["pred"][r] = int(pred[j])
            else:
                rem.append(r)
        assert len(rem) == int(bufs[s].n_surv_host[0])
        return rem, now

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
        out = {"finish": np.zeros(n), "exit_stage": np.full(n, -1), "pred": np.full(n, -1), "launches": [],
               "preemptions": 0, "declined": 0}
        latency = latency or stage_time
        if np.isfinite(slo) and latency is None:
            raise ValueError("a finite SLO needs the exit-level latency table (latency=...)")

        def span(first, last, batch):           # T_{first:last}^{batch}
            return sum(latency(j, batch) for j in range(first, last + 1))
        q: deque = deque()
        nxt = 0
        t0 = time.perf_counter()
        clock = lambda: time.perf_counter() - t0     # noqa: E731
        t = 0.0

        def admit(now):
            nonlocal nxt
            while nxt < n and arrivals[nxt] <= now:
                q.append(nxt)
                nxt += 1

        while nxt < n or q:
            if stage_time is None:
                t = clock()
            admit(t)
            if not q:
                if stage_time is None:
                    while clock() < arrivals[nxt]:
                        pass
                    t = clock()
                else:
                    t = float(arrivals[nxt])
                admit(t)
            act = [q.popleft() for _ in range(min(len(q), self.bmax))]          # B_act = min(N_Q, B_max)
            self._form_batch(pool, [image_of[r] for r in act], act, self.in_act, self.ids_act)
            feat, ids = self.in_act, self.ids_act
            i = 0
            while i < self.n_stages - 1:
                act, t = self._run(i, feat, ids, act, self.act, t, clock, stage_time, out)
                feat, ids = self.act[i].features_out, self.act[i].ids_out       # B_rem parked at the boundary
                while len(act) < self.bmax:
                    admit(t)
                    incr = min(len(q), self.bmax - len(act))                    # B_incr = min(N_Q, B_slack)
                    if incr == 0:
                        break
                    if act and np.isfinite(slo):                                 # SLO-aware preemption criterion
                        t_slack = slo - (t - min(arrivals[r] for r in act))      # Eq. 3, oldest sample of the active batch
                        t_overhead = span(0, i, incr) + span(i + 1, self.n_stages - 1, len(act) + incr)   # Eq. 4
                        if not t_overhead < t_slack:
                            out["declined"] += 1
                            break
                    out["preemptions"] += 1
                    new = [q.popleft() for _ in range(incr)]
                    self._form_batch(pool, [image_of[r] for r in new], new, self.in_new, self.ids_new)
                    nfeat, nids = self.in_new, self.ids_new
                    for j in range(i + 1):                                       # the new batch catches up to exit i
                        new, t = self._run(j, nfeat, nids, new, self.new, t, clock, stage_time, out)
                        nfeat, nids = self.new[j].features_out, self.new[j].ids_out
                        if not new:
                            break
                    if new:                                                      # B_merged = B_rem + B_incr - B_exit
                        n_acc, n_mer = self.m.batch_refill(i + 1, feat, ids, len(act), nfeat, nids, len(new))
                        assert n_acc == len(new) and n_mer == len(act) + len(new)
                        act = act + new
                if not act:
                    break
                i += 1
            if act:
                act, t = self._run(self.n_stages - 1, feat, ids, act, self.act, t, clock, stage_time, out)
                assert not act
        torch.cuda.synchronize()
        return out
