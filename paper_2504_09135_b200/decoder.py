"""Decode-loop helper: B queries x K candidates through disc_step, then disc_resample.

Orchestration only (which kernel is enqueued when); all arithmetic is in the CUDA library.  The
loop never synchronises the host: it runs l_max steps, and rows that finished earlier are skipped
inside the kernel.
"""
from __future__ import annotations

import torch

from .binding import (DiscSet, DiscState, StepOutputs, disc_accept_resample, disc_resample, disc_state_init,
                      disc_step)


class DiscDecoder:
    def __init__(self, s: DiscSet, B: int, K: int, device="cuda", *, want_logq=True, want_logp=True,
                 query_base: int = 0):
        """query_base: global index of this decoder's first query when the queries of a job are
        sharded over several GPUs (shard.shard_queries); it keeps the random-number coordinates of
        a row independent of how the job was split."""
        self.set, self.B, self.K, self.R = s, B, K, B * K
        self.query_base = int(query_base)
        self.device = torch.device(device)
        self.state = DiscState.empty(self.R, self.device)
        self.out = StepOutputs.empty(self.R, self.device, logq=want_logq, logp=want_logp)
        self.seq = torch.empty((self.R, s.l_max), dtype=torch.int32, device=self.device)
        self.res = {"idx": torch.empty(B, dtype=torch.int32, device=self.device),
                    "logz": torch.empty(B, dtype=torch.float32, device=self.device),
                    "status": torch.empty(B, dtype=torch.uint8, device=self.device),
                    "tokens": torch.empty((B, s.l_max), dtype=torch.int32, device=self.device)}

    def reset(self):
        self.seq.fill_(-1)
        disc_state_init(self.set, self.R, state=self.state)

    def step(self, logits: torch.Tensor, step: int, *, seed=0, inv_temperature=1.0, row_base=None) -> StepOutputs:
        row_base = self.query_base * self.K if row_base is None else row_base
        return disc_step(self.set, logits, self.state, inv_temperature=inv_temperature, seed=seed, step=step,
                         row_base=row_base, seq_tokens=self.seq, out=self.out)

    def finish(self, *, seed=0, query_base=None):
        query_base = self.query_base if query_base is None else query_base
        return disc_resample(self.state.logw.view(self.B, self.K), seed=seed, query_base=query_base,
                             seq_tokens=self.seq.view(self.B, self.K, -1), out=self.res)

    def finish_accept_resample(self, *, seed=0, query_base=None):
        """Algorithm 1, lines 11-22 for a decoder created with an even number of candidates per
        query: the first half goes through the accept test in order, the second half are the fresh
        candidates of the K-way draw.  Returns dict(choice, first, logz, status, tokens)."""
        if self.K % 2:
            raise ValueError("finish_accept_resample needs an even number of candidates per query")
        query_base = self.query_base if query_base is None else query_base
        return disc_accept_resample(self.state.logw.view(self.B, self.K), seed=seed, query_base=query_base,
                                    seq_tokens=self.seq.view(self.B, self.K, -1))

    def decode(self, lm, ctx: torch.Tensor, *, seed=0, inv_temperature=1.0, keep_logits=None):
        """Free-running decode: `lm.logits(prev)` gives the [R, V] logits after tokens `prev`.

        ctx: int tensor [B], the context token of each query.  keep_logits: optional list that
        receives each step's logits tensor (for replay)."""
        self.reset()
        prev = ctx.to(self.device, torch.int64).repeat_interleave(self.K)
        for t in range(self.set.l_max):
            logits = lm.logits(prev)
            if keep_logits is not None:
                keep_logits.append(logits)
            o = self.step(logits, t, seed=seed, inv_temperature=inv_temperature)
            prev = torch.where(o.token >= 0, o.token.to(torch.int64), prev)
        return self.finish(seed=seed)

    def replay(self, logits_per_step, *, seed=0, inv_temperature=1.0):
        """Decode over logits that are already resident on the device, one tensor per step."""
        self.reset()
        for t, logits in enumerate(logits_per_step):
            self.step(logits, t, seed=seed, inv_temperature=inv_temperature)
        return self.finish(seed=seed)

    def capture(self, logits_per_step, *, seed=0, inv_temperature=1.0) -> "torch.cuda.CUDAGraph":
        """The same decode recorded once as a CUDA graph (state init, every step, resampling);
        `graph.replay()` then enqueues the whole decode with one call.  The logits tensors, the
        seed and this decoder's buffers are baked in: refill the logits in place between replays.
        Results land in `self.res`, `self.seq` and `self.state` as usual."""
        self.replay(logits_per_step, seed=seed, inv_temperature=inv_temperature)   # first-call set-up outside the capture
        torch.cuda.synchronize(self.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.replay(logits_per_step, seed=seed, inv_temperature=inv_temperature)
        return graph

    def replay_from_host(self, host_logits_per_step, staging: torch.Tensor | None, *, seed=0, inv_temperature=1.0):
        """Same decode with every step's logits coming from pinned host memory, and the result read
        back to the host at the end.  With a staging tensor every step's logits are copied to the
        device first; with staging=None the kernel reads the pinned host memory in place, which
        moves only the rows that are still live across PCIe."""
        self.reset()
        for t, h in enumerate(host_logits_per_step):
            if staging is None:
                self.step(h, t, seed=seed, inv_temperature=inv_temperature)
                continue
            staging.copy_(h, non_blocking=True)
            self.step(staging, t, seed=seed, inv_temperature=inv_temperature)
        r = self.finish(seed=seed)
        return {"idx": r["idx"].cpu(), "tokens": r["tokens"].cpu(), "logz": r["logz"].cpu()}
