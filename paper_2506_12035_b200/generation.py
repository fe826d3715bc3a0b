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
            forced_refresh: Optional[List[torch.Tensor]] = None, stream=None):
        """Enqueues all T steps.  mode "full" runs the full-recompute baseline.  With
        record=True returns per-step host copies (this synchronises every step)."""
        m, B = self.m, self.m.B
        self.hidden.copy_(hidden0, non_blocking=True)
        m.init_cache(self.cache, stream)
        log = []
        k_prev = 0
        for t in range(self.T):
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
            if forced_refresh is not None:
                fr = forced_refresh[t]
                k = fr.shape[1]
                R_out[: B * k].copy_(fr.reshape(-1))
            if record:
                m.get_scores(self.workspace, self.scores, stream)
                torch.cuda.synchronize()
                log.append(dict(
                    t=t, n_active=n_active,
                    active=None if (t == 0 or mode == "full") else active.cpu().numpy().copy(),
                    scores=self.scores.cpu().numpy().copy(),
                    refresh=R_out[: B * k].view(B, k).cpu().numpy().copy(),
                    hidden_out=self.hidden_out.cpu().numpy().copy()))
            m.scatter_rows(self.rows[t], G, self.hidden, stream)
            k_prev = k
        return log
