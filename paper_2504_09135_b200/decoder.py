"""Decode-loop helper: B queries x K candidates through disc_step, then disc_resample.

Orchestration only (which kernel is enqueued when); all arithmetic is in the CUDA library.  The
loop never synchronises the host: it runs l_max steps, and rows that finished earlier are skipped
inside the kernel.

Three ways to take a step: with the exact valid set (disc_step, the default), in the paper's top-M
mode (`top_m=M`: disc_step_topm - the M most probable tokens are verified in the sorted array and the
token is drawn among the verified ones; a row without a valid candidate ends as a dead end), and
from the model's final hidden vectors with the projection fused in (`step_hidden`,
disc_project_step).
"""
from __future__ import annotations

import torch

from .binding import (DiscSet, DiscState, StepOutputs, disc_accept_resample, disc_project_scratch, disc_project_step,
                      disc_resample, disc_state_init, disc_step, disc_step_topm, lib)


class DiscDecoder:
    def __init__(self, s: DiscSet, B: int, K: int, device="cuda", *, want_logq=True, want_logp=True,
                 query_base: int = 0, top_m: int | None = None):
        """query_base: global index of this decoder's first query when the queries of a job are
        sharded over several GPUs (shard.shard_queries); it keeps the random-number coordinates of
        a row independent of how the job was split.
        top_m: None for the exact valid set; M (1..1024) for the paper's top-M mode."""
        self.set, self.B, self.K, self.R = s, B, K, B * K
        self.query_base = int(query_base)
        self.device = torch.device(device)
        self.top_m = None if top_m is None else int(top_m)
        self.cand = self.scratch = None
        if self.top_m is not None:
            need = lib().disc_step_topm_scratch_bytes(self.R, self.top_m)
            if need < 0:
                raise ValueError("top_m: unsupported size")
            self.cand = torch.empty((self.R, self.top_m), dtype=torch.int32, device=self.device)
            self.scratch = torch.empty(int(need), dtype=torch.uint8, device=self.device)
        self._proj = None
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
        if self.top_m is not None:
            return disc_step_topm(self.set, logits, self.state, self.top_m, self.seq, inv_temperature=inv_temperature,
                                  seed=seed, step=step, row_base=row_base, out=self.out, cand=self.cand,
                                  scratch=self.scratch)[0]
        return disc_step(self.set, logits, self.state, inv_temperature=inv_temperature, seed=seed, step=step,
                         row_base=row_base, seq_tokens=self.seq, out=self.out)

    def step_hidden(self, hidden: torch.Tensor, wt: torch.Tensor, step: int, *, seed=0, inv_temperature=1.0,
                    row_base=None) -> StepOutputs:
        """The step from the model's final hidden vectors (bf16 [R, d]) and its vocabulary matrix
        (bf16 [V, d]): the projection runs inside the call and only the pieces of the logits the
        step reads are written (to a buffer this decoder keeps).  Exact valid set only."""
        if self.top_m is not None:
            raise ValueError("step_hidden works with the exact valid set, not in top-M mode")
        row_base = self.query_base * self.K if row_base is None else row_base
        if self._proj is None:
            ld = (self.set.V + 7) // 8 * 8
            self._proj = (torch.empty((self.R, ld), dtype=torch.bfloat16, device=self.device),
                          disc_project_scratch(self.set, self.R, self.device))
        buf, scratch = self._proj
        return disc_project_step(self.set, hidden, wt, self.state, buf, scratch, inv_temperature=inv_temperature,
                                 seed=seed, step=step, row_base=row_base, seq_tokens=self.seq, out=self.out)

    def decode_hidden(self, lm, ctx: torch.Tensor, *, seed=0, inv_temperature=1.0):
        """Free-running decode with the projection fused into every step: `lm.hidden(prev)` gives
        the bf16 [R, d] hidden vectors after tokens `prev`, `lm.projection_rows()` the bf16 [V, d]
        vocabulary matrix."""
        self.reset()
        wt = lm.projection_rows()
        prev = ctx.to(self.device, torch.int64).repeat_interleave(self.K)
        for t in range(self.set.l_max):
            o = self.step_hidden(lm.hidden(prev), wt, t, seed=seed, inv_temperature=inv_temperature)
            prev = torch.where(o.token >= 0, o.token.to(torch.int64), prev)
        return self.finish(seed=seed)

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
