"""T-step generation loop over the C-ABI calls (no arithmetic of its own).

Step 0 is `full_step` (the cache is empty, Section 4.3); step t >= 1 builds
A(t) = G(t) u G(t-1) u R(t) on the device with `build_active` and runs the
cache-aware `step`; R(t) is the refresh set the previous step selected with
G(t) excluded.  After each step the rows of the tokens generated in it are
overwritten in the stack input by caller-supplied rows (the diffusion sampler
of Eq. 3 is outside the hot path).  The loop never reads device memory back,
so a whole generation is enqueued without a host synchronisation.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from .binding import Marche


class Generation:
    def __init__(self, m: Marche, new_sets: Sequence, refresh_ratio: float, sampled_rows: Sequence[torch.Tensor]):
        """new_sets[t]: int32 [B][#G(t)] (array-like); sampled_rows[t]: float [B][#G(t)][D] on the device."""
        self.m = m
        self.ratio = float(refresh_ratio)
        dev = "cuda"
        self.new_sets = [torch.as_tensor(g, dtype=torch.int32).to(dev).contiguous() for g in new_sets]
        self.rows = list(sampled_rows)
        self.T = len(self.new_sets)
        B, S, D = m.B, m.S, m.D
        self.hidden = torch.empty(B, S, D, dtype=torch.float32, device=dev)
        self.hidden_out = torch.zeros(B, S, D, dtype=torch.float32, device=dev)
        self.cache = m.alloc_cache()
        self.workspace = m.alloc_workspace(S)
        self.active_flat = torch.empty(B * S, dtype=torch.int32, device=dev)
        self.refresh_flat = [torch.empty(B * S, dtype=torch.int32, device=dev) for _ in range(2)]
        self.scores = torch.empty(B, S, dtype=torch.float32, device=dev)

    def run(self, hidden0: torch.Tensor, mode: str = "marche", record: bool = False,
            forced_refresh: Optional[List[torch.Tensor]] = None, stream=None, n_steps: Optional[int] = None,
            after_step=None):
        """Enqueues all T steps.  mode "full" runs the full-recompute baseline.  With
        record=True returns per-step host copies (this synchronises every step)."""
        m, B = self.m, self.m.B
        self.hidden.copy_(hidden0, non_blocking=True)
        m.init_cache(self.cache, stream)
        log = []
        k_prev = 0
        for t in range(self.T if n_steps is None else min(n_steps, self.T)):
            G = self.new_sets[t]
            X = self.new_sets[t + 1] if t + 1 < self.T else None
            R_out = self.refresh_flat[t % 2]
            if t == 0 or mode == "full":
                n_active = m.S
                k = m.full_step(self.hidden, self.cache, G, X, self.ratio, self.hidden_out, R_out, self.workspace,
                                stream)
            else:
                R_in = self.refresh_flat[(t - 1) % 2]
                n_active = G.shape[1] + self.new_sets[t - 1].shape[1] + k_prev
                active = self.active_flat[: B * n_active].view(B, n_active)
                m.build_active(G, self.new_sets[t - 1], R_in, k_prev, active, stream)
                k = m.step(self.hidden, self.cache, active, G, X, self.ratio, self.hidden_out, R_out, self.workspace,
                           stream)
            own = None
            if record:                      # the step's own selection, before any forcing
                torch.cuda.synchronize()
                own = R_out[: B * k].view(B, k).cpu().numpy().copy()
            if forced_refresh is not None:
                fr = forced_refresh[t]
                k = fr.shape[1]
                R_out[: B * k].copy_(fr.reshape(-1))
            if record:
                m.get_scores(self.workspace, self.scores, stream)
                torch.cuda.synchronize()
                log.append(dict(
                    t=t, n_active=n_active, refresh_own=own,
                    active=None if (t == 0 or mode == "full") else active.cpu().numpy().copy(),
                    scores=self.scores.cpu().numpy().copy(),
                    refresh=R_out[: B * k].view(B, k).cpu().numpy().copy(),
                    hidden_out=self.hidden_out.cpu().numpy().copy()))
            m.scatter_rows(self.rows[t], G, self.hidden, stream)
            k_prev = k
            if after_step is not None:
                after_step(t)
        return log

    def capture(self, hidden0: torch.Tensor, **run_args) -> "torch.cuda.CUDAGraph":
        """Runs one generation eagerly (first-call set-up of the kernels), then records the same
        generation in a CUDA graph.  graph.replay() re-enqueues all of its launches without any host
        work per launch (about 1 % faster end to end); it reads hidden0 and the sampled rows from the
        same buffers, so new inputs are copied into them before a replay."""
        self.run(hidden0, **run_args)
        torch.cuda.synchronize()
        side = torch.cuda.Stream()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(graph, stream=side):
                self.run(hidden0, **run_args)
        return graph

    # ------------------------------------------------------------------ the paper's own schedule
    def run_in_step(self, hidden0: torch.Tensor, budget: int = 64, period: int = 3, record: bool = False,
                    forced_refresh: Optional[List[Optional[torch.Tensor]]] = None, stream=None,
                    n_steps: Optional[int] = None):
        """Section 4.3 schedule: a full step at t = 0 and every `period`-th step, otherwise
        marche_step_in_step_selection with K = budget - #G - #N refreshing tokens."""
        m, B, S = self.m, self.m.B, self.m.S
        self.hidden.copy_(hidden0, non_blocking=True)
        m.init_cache(self.cache, stream)
        log = []
        for t in range(self.T if n_steps is None else min(n_steps, self.T)):
            G = self.new_sets[t]
            N = self.new_sets[t - 1] if t > 0 else None
            if t % period == 0:
                m.full_step(self.hidden, self.cache, G, None, 0.0, self.hidden_out, None, self.workspace, stream)
                n_active, k, active = S, 0, None
            else:
                n_gn = G.shape[1] + N.shape[1]
                k = min(max(0, budget - n_gn), S - n_gn)
                n_active = n_gn + k
                active = self.active_flat[: B * n_active].view(B, n_active)
                fr = None if forced_refresh is None else forced_refresh[t]
                m.step_in_step_selection(self.hidden, self.cache, G, N, k, fr, self.hidden_out, self.refresh_flat[0],
                                         active, self.workspace, stream)
            if record:
                m.get_scores(self.workspace, self.scores, stream)
                torch.cuda.synchronize()
                log.append(dict(t=t, n_active=n_active, active=None if active is None else active.cpu().numpy().copy(),
                                scores=self.scores.cpu().numpy().copy(),
                                refresh=self.refresh_flat[0][: B * k].view(B, k).cpu().numpy().copy(),
                                hidden_out=self.hidden_out.cpu().numpy().copy()))
            m.scatter_rows(self.rows[t], G, self.hidden, stream)
        return log

    # ------------------------------------------------------------------ two-stage model (Eq. 1, Eq. 2)
    def run_mar(self, tokens0: torch.Tensor, known_sets: Sequence, budget: int = 64, period: int = 3,
                record: bool = False, forced_refresh: Optional[List[Optional[torch.Tensor]]] = None, stream=None,
                n_steps: Optional[int] = None, mode: str = "marche"):
        """Encoder over the known tokens and cache-aware decoder, Section 4.3 schedule: the decoder is
        fully refreshed at t = 0 and every `period`-th step (always with mode "full"), otherwise it
        runs the in-step selection with K = budget - #G - #N.  known_sets[t]: int32 [B][n_known(t)].
        The decoder outputs land in self.hidden_out."""
        m, B, S = self.m, self.m.B, self.m.S
        if not hasattr(self, "known_sets_dev") or len(self.known_sets_dev) != len(known_sets):
            self.known_sets_dev = [torch.as_tensor(k, dtype=torch.int32).to("cuda").contiguous() for k in known_sets]
        self.hidden.copy_(tokens0, non_blocking=True)
        m.init_cache(self.cache, stream)
        log = []
        for t in range(self.T if n_steps is None else min(n_steps, self.T)):
            G = self.new_sets[t]
            N = self.new_sets[t - 1] if t > 0 else None
            Kn = self.known_sets_dev[t]
            if mode == "full" or t % period == 0:
                m.mar_step(True, self.hidden, Kn, self.cache, G, N, 0, None, self.hidden_out, None, None,
                           self.workspace, stream)
                n_active, k, active = S, 0, None
            else:
                n_gn = G.shape[1] + N.shape[1]
                k = min(max(0, budget - n_gn), S - n_gn)
                n_active = n_gn + k
                active = self.active_flat[: B * n_active].view(B, n_active)
                fr = None if forced_refresh is None else forced_refresh[t]
                m.mar_step(False, self.hidden, Kn, self.cache, G, N, k, fr, self.hidden_out, self.refresh_flat[0],
                           active, self.workspace, stream)
            if record:
                m.get_scores(self.workspace, self.scores, stream)
                torch.cuda.synchronize()
                log.append(dict(t=t, n_active=n_active, active=None if active is None else active.cpu().numpy().copy(),
                                scores=self.scores.cpu().numpy().copy(),
                                refresh=self.refresh_flat[0][: B * k].view(B, k).cpu().numpy().copy(),
                                z=self.hidden_out.cpu().numpy().copy()))
            m.scatter_rows(self.rows[t], G, self.hidden, stream)
        return log

    # ------------------------------------------------------------------ host-driven loop
    def alloc_host_buffers(self, hidden0, rows_np, sets_np):
        """Pinned host buffers for run_host: the stack input, per step the sampled rows and
        index sets (inputs) and the output rows / refresh indices (results)."""
        pin = lambda a: torch.as_tensor(a).contiguous().pin_memory()
        B, S, D = self.m.B, self.m.S, self.m.D
        self.h_hidden0 = pin(hidden0)
        self.h_rows = [pin(r) for r in rows_np]
        self.h_sets = [pin(torch.as_tensor(g, dtype=torch.int32)) for g in sets_np]
        self.h_out_rows = [torch.empty(B, g.shape[1], D, dtype=torch.float32).pin_memory() for g in self.h_sets]
        self.h_refresh = torch.empty(B * S, dtype=torch.int32).pin_memory()
        self.max_new = max(g.shape[1] for g in self.h_sets)
        self.staging = torch.empty(self.m.staging_bytes(self.max_new), dtype=torch.uint8, device="cuda")

    def run_host(self, stream=None):
        """The same generation through marche_step_host: every step copies its inputs from
        pinned host memory and its results back.  Returns (h2d_bytes, d2h_bytes) per generation."""
        m, B, D = self.m, self.m.B, self.m.D
        self.hidden.copy_(self.h_hidden0, non_blocking=True)
        h2d = self.h_hidden0.numel() * 4
        d2h = 0
        m.init_cache(self.cache, stream)
        k_prev = 0
        for t in range(self.T):
            prev_rows = self.h_rows[t - 1] if t > 0 else None
            prev_idx = self.h_sets[t - 1] if t > 0 else None
            excl = self.h_sets[t + 1] if t + 1 < self.T else None
            k = m.step_host(t == 0, self.hidden, self.cache, prev_rows, prev_idx, self.h_sets[t], excl,
                            self.refresh_flat[(t - 1) % 2], k_prev, self.ratio, self.hidden_out,
                            self.refresh_flat[t % 2], self.h_out_rows[t], self.h_refresh, self.max_new, self.staging,
                            self.workspace, stream)
            n_new = self.h_sets[t].shape[1]
            n_prev = 0 if prev_idx is None else prev_idx.shape[1]
            n_excl = 0 if excl is None else excl.shape[1]
            h2d += B * n_prev * D * 4 + 4 * B * (n_prev + n_new + n_excl)
            d2h += B * n_new * D * 4 + 4 * B * k
            k_prev = k
        return h2d, d2h
