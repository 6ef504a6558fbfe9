"""Helpers shared by the GPU parity tests: lock-step comparison of disc_step with the oracle."""
import numpy as np
import torch

import oracle
import paper_2504_09135_b200 as disc

TOL = 1e-5          # relative tolerance on log-weights / log-probs; absolute near-tie window (nats)


def logits_to_host(logits: torch.Tensor):
    """Device logits -> (numpy array the oracle reads, oracle dtype code).  Same bytes."""
    if logits.dtype == torch.float32:
        return logits.detach().cpu().numpy(), oracle.F32
    return logits.detach().view(torch.int16).cpu().numpy().view(np.uint16), oracle.BF16


def close(a, b, tol=TOL):
    """|a-b| <= tol*max(1,|b|), with equal infinities and NaN==NaN accepted."""
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    same_special = (np.isnan(a) & np.isnan(b)) | (np.isinf(a) & np.isinf(b) & (np.sign(a) == np.sign(b)))
    with np.errstate(invalid="ignore"):
        ok = np.abs(a - b) <= tol * np.maximum(1.0, np.abs(b))
    return ok | same_special


def assert_near_ties(gpu_tokens, o, sel):
    """The rows in `sel` got a token that differs from the oracle's.  That is accepted only when
    the oracle itself sees a near-tie (and counted): a different token group needs the oracle's
    score of that group within TOL of the winning score; a different token of the same group needs
    the in-group threshold within TOL (relative to the group's mass) of an interval boundary and a
    neighbouring pick.  Rows with NaN/+Inf logits promise no particular token.  Returns the count."""
    idx = np.nonzero(sel)[0]
    n = 0
    for t, i in zip(gpu_tokens, idx):
        if o["status"][i] & 4:
            continue
        if (int(t) >> 3) != (int(o["token"][i]) >> 3):
            assert o["best"][i] - o["alt"][i] < TOL, ("group", i, int(t), int(o["token"][i]), o["best"][i], o["alt"][i])
        else:
            assert o["ingroup_gap"][i] < TOL, ("in-group", i, int(t), int(o["token"][i]), o["ingroup_gap"][i])
        n += 1
    return n


class LockStep:
    """Runs a decode on the GPU and checks every step against the oracle from the same state."""

    def __init__(self, S_gpu, S_cpu, R, device="cuda", rows=None, with_mask=False):
        self.S_gpu, self.S_cpu, self.R = S_gpu, S_cpu, R
        self.device = device
        self.state = disc.disc_state_init(S_gpu, R, device=device)
        self.seq = torch.full((R, S_gpu.l_max), -1, dtype=torch.int32, device=device)
        self.out = disc.StepOutputs.empty(R, device, mask_words=S_gpu.W if with_mask else 0)
        self.rows = np.arange(R) if rows is None else np.asarray(rows)     # rows the oracle checks
        self.near_ties = 0
        self.checked = 0
        self.max_err = 0.0

    def step(self, logits, step: int, seed: int, inv_t: float = 1.0, row_base: int = 0, run=None, oracle_step=None):
        """run: optional callable(state, seq, out) that performs the step on the GPU some other way
        than disc_step (the fused projection, the top-M mode) and returns the logits tensor that
        step used.  oracle_step: optional callable with S_cpu.step's signature that takes its place
        (the top-M mode); rows it ends at a dead end (no token) must end the same way on the GPU."""
        rows = self.rows
        before = {k: getattr(self.state, k).cpu().numpy().copy() for k in ("node", "lo", "hi", "depth", "logw", "done")}
        seq_before = self.seq.cpu().numpy()[rows]
        if run is not None:
            logits = run(self.state, self.seq, self.out)
        else:
            disc.disc_step(self.S_gpu, logits, self.state, inv_temperature=inv_t, seed=seed, step=step,
                           row_base=row_base, seq_tokens=self.seq, out=self.out)
        torch.cuda.synchronize()
        g_tok = self.out.token.cpu().numpy()
        g_status = self.out.status.cpu().numpy()
        after = {k: getattr(self.state, k).cpu().numpy() for k in ("node", "lo", "hi", "depth", "logw", "done")}
        host_logits, dt = logits_to_host(logits[torch.as_tensor(rows, device=logits.device)])
        o = (oracle_step or self.S_cpu.step)(host_logits, dt, seq_before, before["depth"][rows], before["done"][rows],
                                             inv_temperature=inv_t, seed=seed, step=step, row_ids=rows + row_base,
                                             alt_token=g_tok[rows], n_threads=8)
        live = before["done"][rows] == 0
        # rows that ran into a dead end (top-M mode): no token, complete, zero weight, cursor untouched
        stuck = live & (o["token"] < 0)
        if stuck.any():
            assert np.all(g_tok[rows][stuck] == -1) and np.all(g_status[rows][stuck] == o["status"][stuck])
            assert np.all(after["done"][rows][stuck] == 1) and np.all(after["logw"][rows][stuck] == -np.inf)
            for k in ("node", "lo", "hi", "depth"):
                assert np.array_equal(after[k][rows][stuck], before[k][rows][stuck]), k
        self.stuck = getattr(self, "stuck", 0) + int(stuck.sum())
        full_live = live
        live = live & ~stuck
        # rows that were already complete: untouched
        d = ~full_live
        assert np.all(g_tok[rows][d] == -1) and np.all(g_status[rows][d] == disc.ROW_DONE)
        for k in ("node", "lo", "hi", "depth", "logw", "done"):
            assert np.array_equal(after[k][rows][d], before[k][rows][d]), k
        # live rows
        assert np.array_equal(g_status[rows][live], o["status"][live]), "status"
        same = g_tok[rows] == o["token"]
        tie = live & ~same
        if tie.any():
            self.near_ties += assert_near_ties(g_tok[rows][tie], o, tie)
        self.checked += int(live.sum())
        exp_logw = before["logw"][rows].astype(np.float64) + o["log_mass"]
        ok = close(after["logw"][rows][live], exp_logw[live])
        assert ok.all(), ("logw", after["logw"][rows][live][~ok], exp_logw[live][~ok])
        fin = live & np.isfinite(exp_logw)
        if fin.any():
            self.max_err = max(self.max_err, float(np.max(np.abs(after["logw"][rows][fin] - exp_logw[fin])
                                                          / np.maximum(1, np.abs(exp_logw[fin])))))
        agree = live & same
        if self.out.logq is not None:
            assert close(self.out.logq.cpu().numpy()[rows][agree], o["logq"][agree]).all(), "logq"
        if self.out.logp is not None:
            assert close(self.out.logp.cpu().numpy()[rows][agree], o["logp"][agree]).all(), "logp"
        # cursor after the step: ranges and completion from the oracle for the GPU's own prefix
        seq_after = self.seq.cpu().numpy()[rows]
        assert np.array_equal(seq_after[live, :][np.arange(live.sum()), before["depth"][rows][live]], g_tok[rows][live])
        assert np.array_equal(after["depth"][rows][live], before["depth"][rows][live] + 1)
        m, lo, hi, st = self.S_cpu.mask(seq_after[live], after["depth"][rows][live])
        assert np.all(st == 0)
        assert np.array_equal(after["lo"][rows][live], lo) and np.array_equal(after["hi"][rows][live], hi), "range"
        assert np.array_equal(after["done"][rows][live] != 0, ~m.any(axis=1)), "done"
        if self.out.mask is not None:
            mb, _, _, _ = self.S_cpu.mask(seq_before[live], before["depth"][rows][live])
            got = self.out.mask.cpu().numpy().view(np.uint32)[rows][live]
            assert np.array_equal(got, mb), "mask_out"
        return o
