#!/usr/bin/env python
"""Benchmark of the DISC + PPV hot path on the "large" workload (V = 128,256).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload large]

One "step" is one whole decode of the workload's B*K candidates: disc_state_init, one disc_step per
token position (l_max launches; finished rows cost nothing), disc_resample.  The stand-in language
model is outside the timed region: its logits for every position are produced once by a recording
decode and kept resident in HBM (1.05 GB per position at the large workload, so every launch
streams far more than the L2 holds); the timed decodes replay them with the same seed and so
reproduce the same tokens.  Prints ONE JSON line (rank 0).

--impl reference times the CPU oracle (oracle/) as it stands on the host cores, on a bounded sample
of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "disc_decode_tokens_per_s"
UNIT = "tokens/s"


def ncu_traffic_ratio():
    """DRAM bytes per algorithmic byte of disc_step_kernel from the committed ncu summary
    (profiles/disc_step_traffic.txt), or None when the kernel's sources have changed since that
    capture (the figure would describe another kernel)."""
    import hashlib
    try:
        kv = {}
        with open(os.path.join(ROOT, "profiles", "disc_step_traffic.txt")) as f:
            for line in f:
                if ":" in line and not line.startswith("#"):
                    k, v = line.split(":", 1)
                    kv[k.strip()] = v.strip()
        h = hashlib.sha256()
        for name in kv["kernel_sources"].split():
            with open(os.path.join(ROOT, "paper_2504_09135_b200", "csrc", name), "rb") as f:
                h.update(f.read())
        if h.hexdigest() != kv["kernel_sources_sha256"]:
            return None
        return float(kv["dram_bytes_per_algorithmic_byte"])
    except (OSError, KeyError, ValueError):
        return None


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="large", choices=["tiny", "genret", "llm", "large"])
    ap.add_argument("--draws", type=int, default=0, help="override the number of members drawn (profiling)")
    ap.add_argument("--B", type=int, default=0, help="override the number of queries (profiling)")
    ap.add_argument("--K", type=int, default=0, help="override the candidates per query (profiling)")
    ap.add_argument("--positions", type=int, default=0,
                    help="decode only the first P token positions (profiling: bounds the resident logits)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-fused", action="store_true", help="skip the fused projection + step figure")
    ap.add_argument("--cpu-sample-rows", type=int, default=4096)
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._t = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.004)

    def start(self):
        if self.nv is not None:
            self._t = threading.Thread(target=self._run, daemon=True)
            self._t.start()

    def stop(self):
        self._stop.set()
        if self._t is not None:
            self._t.join()
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def popcount_rows(mask):
    """Set bits per row of an int32 [n, W] device tensor (bookkeeping for the byte count only)."""
    import torch
    table = torch.tensor([bin(i).count("1") for i in range(256)], dtype=torch.int32, device=mask.device)
    return table[mask.contiguous().view(torch.uint8).to(torch.int64)].view(mask.shape[0], -1).sum(1)


def logits_to_numpy(t):
    """Logits tensor -> (numpy array of the same bytes, oracle dtype code)."""
    import torch
    if t.dtype == torch.float32:
        return t.detach().cpu().numpy(), 0
    return t.detach().view(torch.int16).cpu().numpy().view(np.uint16), 1


def workload(args):
    from workloads import CONFIGS, scaled
    over = {}
    if args.draws:
        over["n_draws"] = args.draws
    if args.B:
        over["B"] = args.B
    if args.K:
        over["K"] = args.K
    return scaled(args.workload, **over) if over else CONFIGS[args.workload]


def describe(w, N=None):
    s = (f"{w.name}: V={w.V}, {w.n_draws} members drawn (len {w.len_min}-{w.len_max}"
         f"{', EOS-closed' if w.eos else ''}, {w.token_dist} tokens), B={w.B}, K={w.K}, {w.logits} logits, "
         f"stand-in LM d={w.d}")
    if N is not None:
        s += f", |S|={N} after de-duplication"
    return s


# ------------------------------------------------------------------------------------------ ours
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2504_09135_b200 as disc
    from workloads import make_contexts, make_lm_weights, make_set
    from workloads.standin_lm import StandInLM

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the hot path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    # under torchrun the process group is used even with one rank, so that a 1-GPU launch goes
    # through the same barrier / max-over-ranks code as an N-GPU launch
    use_dist = world > 1 or ("RANK" in os.environ and "MASTER_ADDR" in os.environ)
    if use_dist:
        dist.init_process_group("nccl", device_id=dev)
    w = workload(args)
    t_setup = time.time()

    # the constraint set is replicated on every GPU; each rank decodes its own queries
    tok, off = make_set(w)
    G = disc.disc_build_set(tok, off, w.V)
    lm = StandInLM(*make_lm_weights(w), w.logits, dev)
    # weak scaling: the job has world * B queries, rank r decodes the contiguous block
    # shard_queries gives it; row / query coordinates of the random numbers stay global
    from paper_2504_09135_b200.shard import gather_query_results, max_over_ranks, shard_queries, sum_over_ranks
    q_first, q_count = shard_queries(world * w.B, world, rank)
    assert q_count == w.B
    ctx = torch.as_tensor(make_contexts(w, salt=rank), device=dev)
    dec = disc.DiscDecoder(G, w.B, w.K, dev, query_base=q_first)
    seed = 250409135
    L = min(G.l_max, args.positions) if args.positions else G.l_max
    esize = 4 if w.logits == "f32" else 2

    # ---- recording decode: keep every position's logits; count live rows and valid-set sizes
    logits_steps, alive, children = [], [], []
    dec.reset()
    prev = ctx.to(torch.int64).repeat_interleave(w.K)
    mask_buf = torch.empty((dec.R, G.W), dtype=torch.int32, device=dev)
    probe = disc.StepOutputs.empty(dec.R, dev, mask_words=0)
    probe.mask = mask_buf
    for t in range(L):
        logits = lm.logits(prev)
        live = (dec.state.done == 0)
        alive.append(int(live.sum().item()))
        st_copy = dec.state.clone()
        disc.disc_step(G, logits, st_copy, seed=seed, step=t, out=probe)       # mask only, state copy
        c = popcount_rows(mask_buf)
        children.append(int(c[0].item()) if t == 0 else int((c * live).sum().item()))
        o = dec.step(logits, t, seed=seed)
        prev = torch.where(o.token >= 0, o.token.to(torch.int64), prev)
        logits_steps.append(logits)
    first = dec.finish(seed=seed)
    first_tokens = first["tokens"].clone()
    first_logw = dec.state.logw.clone()
    torch.cuda.synchronize()
    assert args.positions or bool(dec.state.done.all()), "decode did not finish within l_max steps"
    del mask_buf, probe
    tokens_per_decode = int(sum(alive))
    job_tokens_per_decode = int(sum_over_ranks(tokens_per_decode, dev))      # all ranks' rows
    launches = [t for t in range(L) if alive[t] > 0]
    alg_bytes = [alive[t] * (w.V * esize + 46) + 4 * children[t] for t in range(L)]

    # ---- stand-in LM projection, timed separately (outside the hot path)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    scratch_logits = torch.empty_like(logits_steps[0])
    lm.logits(prev, out=scratch_logits) if lm.b is None else lm.logits(prev)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(3):
        lm.logits(prev, out=scratch_logits) if lm.b is None else lm.logits(prev)
    e1.record()
    torch.cuda.synchronize()
    lm_ms = e0.elapsed_time(e1) / 3
    del scratch_logits

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- timed region: K whole decodes over the resident logits
    for _ in range(max(args.warmup, 3)):
        dec.replay(logits_steps, seed=seed)
    barrier()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(L)]
          for _ in range(args.steps)]
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.nvtx.range_push("timed")          # lets a profiler restrict itself to the timed region
    t0.record()
    for k in range(args.steps):
        dec.reset()
        for t in range(L):
            ev[k][t][0].record()
            dec.step(logits_steps[t], t, seed=seed)
            ev[k][t][1].record()
        dec.finish(seed=seed)
    t1.record()
    barrier()
    torch.cuda.nvtx.range_pop()
    clocks = sampler.stop()
    total_ms = t0.elapsed_time(t1)
    same_tokens = bool(torch.equal(dec.res["tokens"], first_tokens)) and bool(torch.equal(dec.state.logw, first_logw))
    step_ms = np.array([[ev[k][t][0].elapsed_time(ev[k][t][1]) for t in range(L)] for k in range(args.steps)])
    total_ms = max_over_ranks(total_ms, dev)
    eager_value = args.steps * job_tokens_per_decode / (total_ms * 1e-3)
    eager_ms = total_ms / args.steps
    gpu_launches = args.steps * (1 + L + 1)      # disc_state_init + L x disc_step + disc_resample

    # ---- the same K decodes, each enqueued as one CUDA graph (no events between the launches);
    # this is the headline figure, the eager loop above supplies the per-launch times
    graph = dec.capture(logits_steps, seed=seed)
    for _ in range(3):
        graph.replay()
    barrier()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler2 = ClockSampler(physical_gpu_index(local_rank))
    sampler2.start()
    marks = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    g0.record()
    marks[0].record()
    for k in range(args.steps):
        graph.replay()
        marks[k + 1].record()
    g1.record()
    barrier()
    clocks_graph = sampler2.stop()
    total_ms = g0.elapsed_time(g1)
    per_decode_ms = np.array([marks[k].elapsed_time(marks[k + 1]) for k in range(args.steps)])
    same_tokens = same_tokens and bool(torch.equal(dec.res["tokens"], first_tokens)) \
        and bool(torch.equal(dec.state.logw, first_logw))
    total_ms = max_over_ranks(total_ms, dev)
    value = args.steps * job_tokens_per_decode / (total_ms * 1e-3)
    del graph
    # the job's result: every query's chosen sequence, gathered in query order (outside the timed
    # region; a few KB per rank)
    job_tokens = gather_query_results(dec.res["tokens"], world * w.B)
    assert job_tokens.shape[0] == world * w.B

    # roofline of the dominant kernel (disc_step): algorithmic bytes / device time, launches with live rows
    kern_ms = float(step_ms[:, launches].sum())
    kern_bytes = float(sum(alg_bytes[t] for t in launches)) * args.steps
    achieved = kern_bytes / (kern_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peaks()
    per_step = [{"step": t, "live_rows": alive[t], "ms": round(float(step_ms[:, t].mean()), 4),
                 "gbs": round(alg_bytes[t] / (float(step_ms[:, t].mean()) * 1e-3) / 1e9, 1)} for t in launches]
    roofline = {"bound": "hbm", "kernel": "disc_step_kernel", "achieved": round(achieved, 1), "peak": peak,
                "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}",
                "frac_of_nominal_8TBs": round(achieved / 8000.0, 4),
                "alg_bytes_per_launch": int(kern_bytes / args.steps / len(launches)),
                "avg_launch_ms": round(kern_ms / args.steps / len(launches), 4),
                "traffic": (None if ncu_traffic_ratio() is None
                            else int(ncu_traffic_ratio() * kern_bytes / args.steps / len(launches))),
                "per_step": per_step}

    # ---- end to end: logits start in pinned host memory, result read back to the host
    e2e = None
    host = None
    if not args.no_e2e:
        try:
            host = [torch.empty(l.shape, dtype=l.dtype, pin_memory=True) for l in logits_steps]
        except RuntimeError as err:          # not enough page-locked memory on this host
            host = None
            e2e = {"value": None, "unit": UNIT, "unavailable": f"pinned host buffers: {str(err)[:120]}"}
    if host is not None:
        for h, l in zip(host, logits_steps):
            h.copy_(l)
        staging = torch.empty_like(logits_steps[0])
        torch.cuda.synchronize()
        n_e2e = max(1, min(args.steps, 3))

        def timed_e2e(stage):
            dec.replay_from_host(host, stage, seed=seed)          # warm-up
            barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            wall0 = time.perf_counter()
            a.record()
            for _ in range(n_e2e):
                r = dec.replay_from_host(host, stage, seed=seed)
            b.record()
            barrier()
            wall = time.perf_counter() - wall0
            ms = max_over_ranks(max(a.elapsed_time(b), wall * 1e3), dev)
            assert torch.equal(r["tokens"], first_tokens.cpu())
            return ms, int(sum(v.numel() * v.element_size() for v in r.values()))

        # (a) every position's logits copied to the device, then disc_step; (b) disc_step reads the
        # pinned host tensors in place, so only the rows that are still live cross PCIe
        copy_ms, d2h = timed_e2e(staging)
        inplace_ms, _ = timed_e2e(None)
        h2d_copy = int(sum(h.numel() * h.element_size() for h in host))
        h2d_inplace = int(sum(alive) * w.V * esize)
        tps = lambda ms: round(n_e2e * job_tokens_per_decode / (ms * 1e-3), 1)
        best_inplace = inplace_ms < copy_ms
        e2e = {"value": tps(min(copy_ms, inplace_ms)), "unit": UNIT,
               "h2d_bytes_per_step": h2d_inplace if best_inplace else h2d_copy, "d2h_bytes_per_step": d2h,
               "decodes": n_e2e,
               "how": ("disc_step reads the pinned host logits in place (live rows only cross PCIe)" if best_inplace
                       else "cudaMemcpyAsync of every position's logits into a device buffer, then disc_step"),
               "copy_then_step": {"value": tps(copy_ms), "h2d_bytes_per_step": h2d_copy},
               "read_in_place": {"value": tps(inplace_ms), "h2d_bytes_per_step": h2d_inplace}}
        del host, staging

    # ---- mask-only stress (secondary figure): 65,536 prefixes of the same table
    mask_stress, mask_sample = None, None
    if rank == 0 and w.name == "large":
        from workloads import CONFIGS, make_prefixes
        mw = CONFIGS["mask"]
        prefix, plen = make_prefixes(mw, tok, off)
        mask_sample = (prefix[:4096], plen[:4096])
        pre_d, len_d = torch.as_tensor(prefix, device=dev), torch.as_tensor(plen, device=dev)
        out = disc.disc_mask(G, pre_d, len_d)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(3):
            disc.disc_mask(G, pre_d, len_d, out=out)
        a.record()
        for _ in range(10):
            disc.disc_mask(G, pre_d, len_d, out=out)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / 10
        nbytes = prefix.shape[0] * G.W * 4
        mask_stress = {"prefixes": int(prefix.shape[0]), "ms": round(ms, 4),
                       "prefixes_per_s": round(prefix.shape[0] / (ms * 1e-3), 1),
                       "mask_gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                       "frac": round(nbytes / (ms * 1e-3) / 1e9 / peak, 4)}
        del out
        # the paper's top-M mode (Algorithm 2 as stated) on the recorded logits of the first two
        # positions: selection of the M most probable tokens, their verification in the sorted
        # array, and the whole top-M step, for the M of the paper's ablation
        nv = dec.R
        verify = []
        for pos in range(min(2, L)):
            stp = disc.disc_state_init(G, nv, device=dev)
            seqp = torch.full((nv, G.l_max), -1, dtype=torch.int32, device=dev)
            for t in range(pos):                     # bring the rows to this position with the exact mask
                disc.disc_step(G, logits_steps[t], stp, seed=seed, step=t, seq_tokens=seqp)
            for M in (50, 100, 500, 1000):
                def t_ms(fn, reps=5):
                    fn()
                    torch.cuda.synchronize()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    a.record()
                    for _ in range(reps):
                        fn()
                    b.record()
                    torch.cuda.synchronize()
                    return a.elapsed_time(b) / reps
                cand = disc.disc_topm(logits_steps[pos], w.V, M)
                vo = disc.disc_verify(G, seqp, stp.depth, cand)
                sel_ms = t_ms(lambda: disc.disc_topm(logits_steps[pos], w.V, M))
                ver_ms = t_ms(lambda: disc.disc_verify(G, seqp, stp.depth, cand, out=vo))
                outp = disc.StepOutputs.empty(nv, dev)
                step_ms = t_ms(lambda: disc.disc_step_topm(G, logits_steps[pos], stp.clone(), M, seqp.clone(),
                                                           seed=seed, step=pos, out=outp))
                verify.append({"position": pos, "rows": nv, "M": M, "select_ms": round(sel_ms, 4),
                               "verify_ms": round(ver_ms, 4), "step_topm_ms": round(step_ms, 4),
                               "candidates_per_s": round(nv * M / (ver_ms * 1e-3), 1),
                               "valid_fraction": round(float(vo["valid"].float().mean().item()), 4),
                               "dead_end_rows": int((outp.status == 1).sum().item())})
        mask_stress["verify_top_m"] = verify

    # ---- a whole decode in the paper's top-M mode next to the exact-mask decode (secondary figure)
    topm_decode = None
    if rank == 0 and w.name == "large" and not args.no_fused:
        try:
            topm_decode = top_m_decode(disc, G, lm, ctx, w, dev, L, seed)
        except Exception as e:                     # a secondary figure never fails the line
            topm_decode = {"error": repr(e)[:200]}
        torch.cuda.empty_cache()

    # ---- the projection fused with the step (secondary figure): a free-running decode per variant,
    # an event pair around every position; the unfused variant is torch's matmul + disc_step
    fused = None
    if rank == 0 and w.logits == "bf16" and not args.no_fused:
        fused = fused_projection(disc, G, lm, ctx, w, dev, L, seed)

    # ---- CPU baseline: the oracle as it stands, on a bounded sample, rank 0 at N = 1 only
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        seq = dec.seq.cpu().numpy()
        cpu = cpu_baseline(w, tok, off, [l[:args.cpu_sample_rows] for l in logits_steps], seq[:args.cpu_sample_rows],
                           seed, mask_sample)

    if rank == 0:
        line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": round(total_ms / args.steps, 4),
                "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
                "data": "synthetic", "impl": "ours",
                "config": {"workload": describe(w, G.N), "tokens_per_decode": tokens_per_decode,
                           "positions": L, "logits_bytes_per_decode": int(sum(alive) * w.V * esize),
                           "l2": "inputs larger than L2: every launch streams its own logits buffer "
                                 f"({dec.R * w.V * esize / 1e6:.0f} MB), no flush needed",
                           "parallelism": f"replicated set, queries sharded over {world} GPU(s), no collective"},
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": gpu_launches,
                "clocks": clocks_graph,
                "ms_per_step_median": round(float(np.median(per_decode_ms)), 4),
                "ms_per_step_best": round(float(per_decode_ms.min()), 4),
                "timed": "each step = one decode (state init, one disc_step per position, resampling) replayed as "
                         "one CUDA graph",
                "eager": {"value": round(eager_value, 1), "ms_per_step": round(eager_ms, 4),
                          "note": "same decode as individual launches with a CUDA event pair around each disc_step "
                                  "(source of the roofline's per-launch times)", "clocks": clocks},
                "deterministic_replay": same_tokens,
                "lm_projection_ms_per_position": round(lm_ms, 3), "mask_stress": mask_stress,
                "fused_projection": fused, "top_m_decode": topm_decode,
                "set": {"members": G.N, "entries": G.E, "index_nodes": G.n_nodes,
                        "device_mb": round(G.device_bytes / 1e6, 1), "build_s": round(G.build_seconds, 3)},
                "setup_s": round(time.time() - t_setup, 1)}
        print(json.dumps(line))
    G.close()
    if use_dist:
        dist.destroy_process_group()


def top_m_decode(disc, G, lm, ctx, w, dev, L, seed, M=50, bonus=8.0, reps=5):
    """Secondary figure: a whole decode in the paper's top-M mode (DiscDecoder(top_m=M)), next to the
    exact-mask decode of the same logits.  The stand-in model knows nothing of the set, so its top-M
    tokens are almost never valid after the first position; a model trained for the task puts its
    mass on valid tokens.  The logits used here stand in for such a model: the stand-in's logits with
    `bonus` added to every valid next token (the valid sets come from disc_mask, outside the timed
    region).  Both decodes replay the same recorded logits as one CUDA graph each."""
    import torch
    R = w.R
    rec = disc.DiscDecoder(G, w.B, w.K, dev, top_m=M)
    rec.reset()
    prev = ctx.to(dev, torch.int64).repeat_interleave(w.K)
    shifts = torch.arange(32, device=dev, dtype=torch.int32)
    steps = []
    for t in range(L):
        z = lm.logits(prev)
        m = disc.disc_mask(G, rec.seq, rec.state.depth)["mask"]
        for r0 in range(0, R, 512):                               # in slices: the unpacked bits are 32 x the mask
            bits = ((m[r0:r0 + 512].unsqueeze(-1) >> shifts) & 1).reshape(min(512, R - r0), -1)[:, :w.V]
            z[r0:r0 + 512] += (bits * bonus).to(z.dtype)
        steps.append(z)
        o = rec.step(z, t, seed=seed)
        prev = torch.where(o.token >= 0, o.token.to(torch.int64), prev)
    rec.finish(seed=seed)
    torch.cuda.synchronize()
    tokens_topm = int((rec.seq >= 0).sum().item())
    dead = int(torch.isinf(rec.state.logw).sum().item())

    def timed(decoder):
        graph = decoder.capture(steps, seed=seed)
        for _ in range(2):
            graph.replay()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            graph.replay()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / reps

    ms_topm = timed(rec)
    exact = disc.DiscDecoder(G, w.B, w.K, dev)
    ms_exact = timed(exact)
    tokens_exact = int((exact.seq >= 0).sum().item())
    return {"M": M, "bonus_on_valid_tokens": bonus,
            "top_m": {"ms_per_decode": round(ms_topm, 4), "tokens_per_decode": tokens_topm,
                      "tokens_per_s": round(tokens_topm / (ms_topm * 1e-3), 1), "dead_end_rows": dead},
            "exact_mask": {"ms_per_decode": round(ms_exact, 4), "tokens_per_decode": tokens_exact,
                           "tokens_per_s": round(tokens_exact / (ms_exact * 1e-3), 1)},
            "note": "same logits for both decodes (stand-in logits + bonus on the valid next tokens of the top-M "
                    "decode's own prefixes); each decode replayed as one CUDA graph"}


def fused_projection(disc, G, lm, ctx, w, dev, L, seed, reps=3):
    """Per-position device time of (a) torch matmul + disc_step and (b) disc_project_step, each over
    its own free-running decode of the workload, from the same contexts."""
    import torch
    R = w.R
    wt = lm.projection_rows()
    scratch = disc.disc_project_scratch(G, R, dev)
    logits = torch.empty((R, w.V), dtype=torch.bfloat16, device=dev)
    seq = torch.empty((R, G.l_max), dtype=torch.int32, device=dev)
    out = disc.StepOutputs.empty(R, dev)
    peak_tf = peak_sus = None
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            peaks = json.load(f)
            peak_tf = float(peaks.get("bf16_tflops", 0)) or None
            peak_sus = float(peaks.get("bf16_tflops_sustained", 0)) or None

    def decode(fused_path):
        ms = np.zeros(L)
        live = np.zeros(L, dtype=np.int64)
        state = disc.disc_state_init(G, R, device=dev)
        seq.fill_(-1)
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        for t in range(L):
            live[t] = int((state.done == 0).sum().item())
            h = lm.hidden(prev)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            if fused_path:
                disc.disc_project_step(G, h, wt, state, logits, scratch, seed=seed, step=t, seq_tokens=seq, out=out)
            else:
                torch.matmul(h, lm.W, out=logits)
                disc.disc_step(G, logits, state, seed=seed, step=t, seq_tokens=seq, out=out)
            b.record()
            torch.cuda.synchronize()
            ms[t] = a.elapsed_time(b)
            prev = torch.where(out.token >= 0, out.token.to(torch.int64), prev)
        if fused_path:
            disc.disc_project_check(scratch)
        return ms, live

    res = {}
    for name, fp in (("unfused", False), ("fused", True)):
        decode(fp)                                           # warm-up
        runs = [decode(fp) for _ in range(reps)]
        ms = np.mean([r[0] for r in runs], axis=0)
        res[name] = {"ms_per_position": [round(float(x), 4) for x in ms], "ms_per_decode": round(float(ms.sum()), 3),
                     "live_rows": [int(x) for x in runs[0][1]]}
    flop = 2.0 * R * w.V * lm.d
    later = res["fused"]["ms_per_position"][1:] or res["fused"]["ms_per_position"]
    tf = flop / (float(np.mean(later)) * 1e-3) / 1e12
    res["flop_per_position"] = flop
    res["fused_tflops_after_position_0"] = round(tf, 1)
    res["roofline"] = {"bound": "tensor", "kernel": "disc_project_pair_kernel (+ tile flags + step)", "achieved": round(tf, 1),
                       "peak": peak_tf, "unit": "TFLOP/s", "frac": None if not peak_tf else round(tf / peak_tf, 4),
                       "peak_kind": "of measured (cuBLAS bf16 burst)" if peak_tf else "unavailable",
                       # the positions are timed one after the other inside decodes that keep the GPU at its
                       # power cap, which is what the sustained figure of the same library GEMM describes
                       "peak_sustained": peak_sus, "frac_of_sustained": None if not peak_sus else round(tf / peak_sus, 4),
                       "traffic": None}
    # end to end through the fused call: every position's hidden vectors start in pinned host memory
    # (R x d bf16 instead of R x V logits), the chosen sequences are read back at the end
    try:
        hid = []
        state = disc.disc_state_init(G, R, device=dev)
        seq.fill_(-1)
        prev = ctx.to(torch.int64).repeat_interleave(w.K)
        for t in range(L):                      # record the hidden vectors of one decode
            h = lm.hidden(prev)
            hid.append(torch.empty(h.shape, dtype=h.dtype, pin_memory=True).copy_(h))
            disc.disc_project_step(G, h, wt, state, logits, scratch, seed=seed, step=t, seq_tokens=seq, out=out)
            prev = torch.where(out.token >= 0, out.token.to(torch.int64), prev)
        torch.cuda.synchronize()
        hbuf = torch.empty_like(lm.hidden(prev))
        res_idx = {"idx": torch.empty(w.B, dtype=torch.int32, device=dev),
                   "logz": torch.empty(w.B, dtype=torch.float32, device=dev),
                   "status": torch.empty(w.B, dtype=torch.uint8, device=dev),
                   "tokens": torch.empty((w.B, G.l_max), dtype=torch.int32, device=dev)}

        def host_decode():
            disc.disc_state_init(G, R, state=state)
            seq.fill_(-1)
            toks = 0
            for t in range(L):
                hbuf.copy_(hid[t], non_blocking=True)
                disc.disc_project_step(G, hbuf, wt, state, logits, scratch, seed=seed, step=t, seq_tokens=seq, out=out)
            r = disc.disc_resample(state.logw.view(w.B, w.K), seed=seed, seq_tokens=seq.view(w.B, w.K, -1), out=res_idx)
            return r["tokens"].cpu(), r["idx"].cpu()

        host_decode()
        torch.cuda.synchronize()
        n_rep = 3
        t0 = time.perf_counter()
        for _ in range(n_rep):
            host_decode()
        torch.cuda.synchronize()
        wall = (time.perf_counter() - t0) / n_rep
        tokens = int(sum(res["fused"]["live_rows"]))
        res["e2e_from_host_hidden"] = {"value": round(tokens / wall, 1), "unit": UNIT, "ms_per_decode": round(wall * 1e3, 3),
                                       "h2d_bytes_per_step": int(sum(h.numel() * h.element_size() for h in hid)),
                                       "d2h_bytes_per_step": int(w.B * (G.l_max + 1) * 4),
                                       "how": "hidden vectors copied from pinned host memory before every "
                                              "disc_project_step; the projection matrix is resident; wall clock"}
    except RuntimeError as err:
        res["e2e_from_host_hidden"] = {"value": None, "unavailable": str(err)[:120]}
    res["note"] = ("each variant decodes on its own (the projections differ in the last bit of a few logits, so the "
                   "sampled sequences may part); the projection computes every row, complete or not, in both variants")
    return res


# ----------------------------------------------------------------------------- oracle on the host
def cpu_baseline(w, tok, off, logits_rows, seq, seed, mask_sample=None):
    """Times oracle.step on the sampled rows over every position (teacher-forced on the GPU's own
    tokens, so each call does the work of the corresponding disc_step rows)."""
    import oracle
    cores = os.cpu_count() or 1
    t0 = time.time()
    S = oracle.OracleSet(tok, off, w.V)
    build_s = time.time() - t0
    n = seq.shape[0]
    lens = (seq >= 0).sum(1)
    host = [logits_to_numpy(l) for l in logits_rows]

    def run(rows, n_threads):
        toks, secs = 0, 0.0
        for t, (hl, dt) in enumerate(host):
            done = (lens[:rows] <= t).astype(np.uint8)
            if done.all():
                break
            a = time.perf_counter()
            S.step(hl[:rows], dt, seq[:rows], np.full(rows, t, np.int32), done, seed=seed, step=t, n_threads=n_threads)
            secs += time.perf_counter() - a
            toks += int((done == 0).sum())
        return toks, secs

    toks_all, secs_all = run(n, cores)
    n1 = max(1, n // 16)
    toks_1, secs_1 = run(n1, 1)
    out = {"value": round(toks_all / secs_all, 1), "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"first {n} of {w.R} rows, all positions ({toks_all} tokens, {secs_all:.1f} s)",
           "value_1_thread": round(toks_1 / secs_1, 1), "sample_1_thread": f"first {n1} rows ({secs_1:.1f} s)",
           "trie_build_s": round(build_s, 1)}
    if mask_sample is not None:      # the mask stress on one host thread (the oracle's mask walk is serial)
        a = time.perf_counter()
        S.mask(*mask_sample)
        out["mask_prefixes_per_s_1_thread"] = round(mask_sample[1].shape[0] / (time.perf_counter() - a), 1)
        out["mask_sample"] = f"first {mask_sample[1].shape[0]} of the 65,536 prefixes"
    return out


def run_reference(args):
    """The oracle as the reference arm: rank 0 only; each step decodes a bounded sample of the
    workload (the first rows) on the host cores.  The logits come from the stand-in LM (on the GPU
    when there is one) and are outside the timed region, as in the other arm."""
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if rank != 0:
        return
    import torch

    import oracle
    from workloads import make_contexts, make_lm_weights, make_set
    from workloads.standin_lm import StandInLM
    w = workload(args)
    cores = os.cpu_count() or 1
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    tok, off = make_set(w)
    t0 = time.time()
    S = oracle.OracleSet(tok, off, w.V)
    build_s = time.time() - t0
    lm = StandInLM(*make_lm_weights(w), w.logits, dev)
    rows = min(w.R, max(w.K, (min(args.cpu_sample_rows, 512) // w.K) * w.K))
    B = rows // w.K
    ctx = make_contexts(w)[:B]
    seed = 250409135

    def decode():
        seq = np.full((rows, S.l_max), -1, np.int32)
        done = np.zeros(rows, np.uint8)
        logw = np.zeros(rows, np.float64)
        prev = np.repeat(ctx, w.K).astype(np.int64)
        secs, toks = 0.0, 0
        for t in range(S.l_max):
            if done.all():
                break
            hl, dt = logits_to_numpy(lm.logits(torch.as_tensor(prev)))
            a = time.perf_counter()
            o = S.step(hl, dt, seq, np.full(rows, t, np.int32), done, seed=seed, step=t, n_threads=cores)
            secs += time.perf_counter() - a
            live = done == 0
            toks += int(live.sum())
            seq[live, t] = o["token"][live]
            logw[live] += o["log_mass"][live]
            prev[live] = o["token"][live]
            done = np.where(live, o["done"], done).astype(np.uint8)
        a = time.perf_counter()
        oracle.resample(logw.reshape(B, w.K).astype(np.float32), seed=seed)
        secs += time.perf_counter() - a
        return toks, secs

    for _ in range(min(args.warmup, 1)):
        decode()
    toks = secs = 0
    for _ in range(args.steps):
        a, b = decode()
        toks += a
        secs += b
    value = toks / secs
    line = {"metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": min(args.warmup, 1), "ms_per_step": round(secs / args.steps * 1e3, 3),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "impl": "reference",
            "config": {"workload": describe(w, S.N), "positions": S.l_max},
            "cpu_baseline": {"value": round(value, 1), "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"first {rows} of {w.R} rows per step, all positions",
                             "trie_build_s": round(build_s, 1)},
            "e2e": {"value": round(value, 1), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


if __name__ == "__main__":
    a = parse_args()
    if a.impl == "reference":
        run_reference(a)
    else:
        run_ours(a)
