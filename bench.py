#!/usr/bin/env python
"""Throughput of the WISV edge-side verifier round on B200, next to its CPU oracle.

  python bench.py --gpus N --steps K --warmup W [--workload NAME] [--impl reference]

One step = one whole verification round (pack -> LM head -> decision head ->
merge/scan) over one batch of seeded synthetic windows.  The default workload is
the Llama-3-8B-shaped batch-1 verifier (B=1, K=8, H=4096, V=128256).  Prints one
JSON line: verified draft tokens/s with inputs resident in HBM (`value`), the
same through the host-buffer entry point with copies inside the timed region
(`e2e`), the roofline of the dominant kernel (LM head) from CUDA events recorded
by the library around that kernel, and the oracle timed on the host cores.
With N > 1 (torchrun) every rank verifies its own batch on its own GPU (requests
are independent: no data-path collective) and the job-wide rate is reported.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import gen  # noqa: E402

METRIC = "verified draft tokens/s at 8B shape (B×K); % of HBM or bf16 TC roofline"
UNIT = "draft tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


# DRAM traffic of the LM-head kernel per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the
# ncu captures summarised under profiles/, keyed by workload, with the hash of the kernel sources the
# capture was taken on: a kernel that has changed since reports traffic = null.
SINGLE_CTA_SOURCES = ("wisv_gemm.cuh", "wisv_ptx.cuh")
CTA_PAIR_SOURCES = ("wisv_gemm2.cuh", "wisv_gemm.cuh", "wisv_ptx.cuh")
NCU_TRAFFIC = {
    # LM-head and decision-head CTAs in one launch, 9 window rows: 1.0642 GB read + 3.8-4.4 MB written per launch
    "8b_b1": {"bytes": 1068300000, "files": SINGLE_CTA_SOURCES, "kernel_hash": "7de628215d9b7ebf"},
    # CTA pairs (one row block of 144) + decision-head clusters: 1.0758 GB read + 4.6-5.4 MB written per launch
    "8b_b16": {"bytes": 1080800000, "files": CTA_PAIR_SOURCES, "kernel_hash": "901db3c2a09c4c22"},
    # CTA pairs (two teams, row blocks of 144) + a decision-head cluster: 1.1039 GB read + 3.9-4.7 MB written per launch
    "8b_b32": {"bytes": 1108200000, "files": CTA_PAIR_SOURCES, "kernel_hash": "901db3c2a09c4c22"},
    # CTA pairs (three teams, row blocks of 192) + decision-head clusters: 1.1218 GB read + 3.7-3.9 MB written per launch
    "8b_b64": {"bytes": 1125600000, "files": CTA_PAIR_SOURCES, "kernel_hash": "901db3c2a09c4c22"},
    # CTA pairs (34 row blocks of 256, two raster groups): 4.48-4.93 GB read + 139-142 MB written (the partials) per
    # launch in this capture; what falls out of L2 depends on where the buffers land, and other captures of the same
    # plan read 2.3-5.4 GB
    "8b_b512": {"bytes": 4844000000, "files": CTA_PAIR_SOURCES, "kernel_hash": "901db3c2a09c4c22"},
}


def kernel_source_hash(files=SINGLE_CTA_SOURCES):
    """sha256 of the kernel sources with comments and white space removed (a reworded comment is not another kernel)."""
    import hashlib
    import re
    h = hashlib.sha256()
    for name in files:
        with open(os.path.join(ROOT, "paper_2604_17701_b200", "csrc", name), "r", encoding="utf-8") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(re.sub(r"\s+", "", text).encode("utf-8"))
    return h.hexdigest()[:16]


def captured_traffic(workload):
    rec = NCU_TRAFFIC.get(workload)
    if not rec:
        return None
    try:
        return rec["bytes"] if rec["kernel_hash"] == kernel_source_hash(rec["files"]) else None
    except Exception:
        return None


class Ranks:
    """Rendezvous, barrier and max-over-ranks for the one-process-per-GPU launch (plain no-ops at N = 1)."""

    def __init__(self, world, backend="nccl", device=None):
        self.world = world
        self.device = device
        self.dist = None
        if world > 1:
            import torch
            import torch.distributed as dist
            kw = {"device_id": torch.device(device)} if backend == "nccl" else {}
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max(self, x):
        if self.dist is None:
            return float(x)
        import torch
        t = torch.tensor([float(x)], dtype=torch.float64, device=self.device if self.device else "cpu")
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def all_gather(self, gathered, part):
        """gathered[g] = rank g's part (gathered: [world, ...] contiguous)."""
        if self.dist is None:
            gathered[0].copy_(part)
        elif self.dist.get_backend() == "nccl":
            self.dist.all_gather_into_tensor(gathered, part)
        else:
            self.dist.all_gather(list(gathered.unbind(0)), part)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def aggregate(world, units_per_rank, ms_per_step):
    """Whole-job rate: every rank processed units_per_rank in the (max-over-ranks) step time."""
    return world * units_per_rank / (ms_per_step * 1e-3)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clocks / throttle reasons sampled while the timed regions run."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.idx = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "100"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
            # the first sample takes a moment: wait for it (bounded) so that short regions are covered too
            t0 = time.time()
            while time.time() - t0 < 3.0 and os.path.getsize(self.f.name) == 0:
                time.sleep(0.02)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is not None:
            self.p.terminate()
            try:
                self.p.wait(timeout=5)
            except Exception:
                self.p.kill()
        try:
            self.f.flush()
            self.f.seek(0)
            sm, mx, reasons = [], [], set()
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            for line in self.f.read().splitlines():
                c = [x.strip() for x in line.split(",")]
                if len(c) < 9:
                    continue
                try:
                    sm.append(float(c[1]))
                    mx.append(float(c[2]))
                except ValueError:
                    continue
                for n, v in zip(names, c[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            if sm:
                out = {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                       "samples": len(sm)}
        finally:
            self.f.close()
            try:
                os.unlink(self.f.name)
            except OSError:
                pass
        return out


def pick_requests(case, n):
    """First, last and a seeded fill: a bounded sample of whole requests."""
    B = case["cfg"].B
    if n >= B:
        return list(range(B))
    picks = {0, B - 1}
    rest = [int(b) for b in np.random.default_rng(0).permutation(B) if b not in picks]
    return sorted(list(picks) + rest[:max(0, n - len(picks))])


def subset_case(case, reqs):
    cfg = case["cfg"]
    k_len = case["k_len"][reqs]
    tok = np.concatenate([np.arange(case["k_off"][b], case["k_off"][b + 1]) for b in reqs]).astype(np.int64)
    row = np.concatenate([np.arange(case["row_off"][b], case["row_off"][b + 1]) for b in reqs]).astype(np.int64)
    k_off, row_off = gen.row_offsets(k_len)
    sub = dict(case)
    sub.update(cfg=cfg.with_(B=len(reqs)), k_len=k_len, k_off=k_off, row_off=row_off, T=int(k_off[-1]),
               R=int(row_off[-1]), target_hidden=case["target_hidden"][row], draft_tokens=case["draft_tokens"][tok],
               csi=case["csi"][reqs])
    if case["sel_off"] is not None:
        sel = np.concatenate([np.arange(case["sel_off"][b], case["sel_off"][b + 1]) for b in reqs]).astype(np.int64)
        cnt = [int(case["sel_off"][b + 1] - case["sel_off"][b]) for b in reqs]
        sub.update(sel_off=np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32), sel_pos=case["sel_pos"][sel],
                   draft_hidden=case["draft_hidden"][sel])
    else:
        sub.update(draft_hidden=case["draft_hidden"][tok])
    for k in ("draft_q", "uniforms"):
        if case[k] is not None:
            sub[k] = case[k][tok]
    return sub


def oracle_round(case):
    """One verification round of the CPU oracle on a case (test infrastructure, timed as the baseline)."""
    import oracle
    cfg = case["cfg"]
    act = {"relu": oracle.ACT_RELU, "gelu": oracle.ACT_GELU}[cfg.act]
    return oracle.verify(lm_head_bits=case["lm_head"], W1_bits=case["W1"], b1=case["b1"], w2=case["w2"],
                         b2=float(case["b2"]), act=act, tau=cfg.tau, k_len=case["k_len"],
                         target_hidden=case["target_hidden"], draft_tokens=case["draft_tokens"],
                         draft_hidden=case["draft_hidden"], csi=case["csi"], sel_off=case["sel_off"],
                         sel_pos=case["sel_pos"], draft_q=case["draft_q"], uniforms=case["uniforms"])


def oracle_sample_size(case, rows_budget):
    """Requests whose window rows add up to about rows_budget."""
    mean_rows = case["R"] / max(1, case["cfg"].B)
    return max(1, min(case["cfg"].B, int(rows_budget / mean_rows)))


def workload_config(name, rank=0):
    cfg = gen.config(name)
    return cfg.with_(seed=cfg.seed + 1000 * rank) if rank else cfg


def config_block(cfg, case, extra=None):
    d = {"workload": cfg.name, "B": cfg.B, "K": cfg.K if cfg.K_hi == 0 else "U{%d..%d}" % (cfg.K_lo, cfg.K_hi),
         "H": cfg.H, "V": cfg.V, "H_d": cfg.H_d, "d_J": cfg.d_J, "d_c": cfg.d_c, "mode": cfg.mode,
         "accept": "stochastic" if cfg.stochastic else "greedy", "act": cfg.act, "tau": cfg.tau,
         "match_rate": cfg.match_rate, "window_rows": case["R"], "draft_tokens": case["T"],
         "l2": "no flush: every step streams the 1.05 GB bf16 LM head, far larger than the 126 MB L2"}
    if extra:
        d.update(extra)
    return d


# ------------------------------------------------------------------------------------- reference arm

def run_reference(args, rank, world):
    """Time the CPU oracle as it stands on the host cores (rank 0 only)."""
    if rank != 0:
        return
    import oracle
    from gen import cases
    cfg = workload_config(args.workload)
    try:
        import torch
        prep_dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    except Exception:
        prep_dev = "cpu"
    # input preparation only (which draft tokens are forced to match); the timed work below is the CPU oracle
    case = cases.make_case(cfg, lambda w, h: cases.library_ref_argmax(w, h, device=prep_dev))
    n_req = oracle_sample_size(case, args.oracle_rows)
    sub = subset_case(case, pick_requests(case, n_req))
    for _ in range(args.warmup):
        oracle_round(sub)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_round(sub)
    dt = (time.perf_counter() - t0) / max(1, args.steps)
    value = sub["T"] / dt
    sample = "%d of %d requests (%d window rows, %d draft tokens) per step" % (n_req, cfg.B, sub["R"], sub["T"])
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_block(cfg, case, {"sampled_requests": n_req}),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------- CUDA arm

NOMINAL_PEAKS = {"hbm_gbs": 7700.0, "bf16_tflops": 2250.0}       # HGX B200 data-sheet figures (dense bf16)
# further configurations of the same 8B model: 144 rows (one row block on CTA pairs, still bound by HBM), then the
# tensor-bound ones
DEFAULT_LEGS = ("8b_b16", "8b_b64", "8b_sh256", "8b_b512")
SHM_DIR = "/dev/shm"


def shared_weights(cfg, rank, ranks):
    """Model weights of a workload; with several ranks the LM head (1 GB at 8B shapes) is generated once.

    Rank 0 writes it to a file in shared memory named after its shape and seed, the other ranks map that file
    instead of all regenerating it at once on the same host cores; rank 0 removes the file when the job ends.
    Returns (weights, path or None).
    """
    if ranks.world == 1 or cfg.weight_seed < 0:         # (no model seed of its own: every rank's batch seed makes its model)
        return gen.make_weights(cfg), None
    ws = cfg.weight_seed if cfg.weight_seed >= 0 else cfg.seed
    path = os.path.join(SHM_DIR, "wisv_lm_head_%dx%d_seed%d_%s.npy" % (cfg.V, cfg.H, ws, os.environ.get("MASTER_PORT", "0")))
    w = None
    if rank == 0:
        w = gen.make_weights(cfg)
        tmp = path + ".tmp%d" % os.getpid()
        np.save(tmp, w["lm_head"])
        os.replace(tmp + ".npy" if not tmp.endswith(".npy") else tmp, path)
    ranks.barrier()
    if rank != 0:
        w = gen.make_weights(cfg, lm_head=np.load(path, mmap_mode="r"))
    ranks.barrier()
    return w, (path if rank == 0 else None)


def device_weights(w, dev):
    import torch
    out = {k: torch.from_numpy(np.ascontiguousarray(w[k]).view(np.int16)).view(torch.bfloat16).to(dev)
           for k in ("lm_head", "W1")}
    out.update({k: torch.from_numpy(np.ascontiguousarray(w[k])).to(dev) for k in ("b1", "w2")})
    return out


def region_stats(ms_list):
    return {"median": float(statistics.median(ms_list)), "min": float(min(ms_list)), "max": float(max(ms_list)),
            "regions": len(ms_list)}


def decision_stats(case, out, cfg):
    """What the round decided, from the device outputs: accepted lengths, |S| histogram, closed-form mean."""
    A = out.accept_len.cpu().numpy().astype(np.int64)
    nm = out.n_mismatch.cpu().numpy().astype(np.int64)
    d = {"mean_accept_len": float(A.mean()), "accepted_tokens": int(A.sum()),
         "m_r_histogram": np.bincount(nm, minlength=1).tolist(), "mean_m_r": float(nm.mean())}
    if cfg.K_hi == 0 and cfg.mode == "FH" and not cfg.stochastic and cfg.B >= 32:
        # positions are i.i.d. by construction of the synthetic batch: each one lets the window continue with
        # probability a = 1 - P(candidate and head probability >= tau), so E[A] = a (1 - a^K) / (1 - a)
        k = cfg.K
        am = out.argmax.cpu().numpy()
        rows = np.repeat(case["row_off"][:-1], case["k_len"]) + (np.arange(case["T"]) - np.repeat(case["k_off"][:-1], case["k_len"]))
        stop = (case["draft_tokens"] != am[rows]) & (out.head_prob.cpu().numpy() >= cfg.tau)
        a = 1.0 - float(stop.mean())
        expect = float(k) if a >= 1.0 else a * (1 - a ** k) / (1 - a)
        sigma = float(A.std() / np.sqrt(len(A)))
        d["closed_form_accept_len"] = {"per_position_continue_prob": a, "expected": expect, "measured": float(A.mean()),
                                       "sigma_of_mean": sigma, "within_3_sigma": bool(abs(A.mean() - expect) <= 3 * sigma + 1e-9)}
    return d


def oracle_check(case, out, cfg, rows_budget, seconds, repeat):
    """The CPU oracle on a bounded sample of whole requests: its rate, and what it says about the device results."""
    import oracle
    n_req = oracle_sample_size(case, rows_budget)
    reqs = pick_requests(case, n_req)
    sub = subset_case(case, reqs)
    t0 = time.perf_counter()
    ref = oracle_round(sub)
    rounds = 1
    while repeat and (time.perf_counter() - t0) < seconds and rounds < 200:
        oracle_round(sub)                               # small workloads: repeat to reach the time budget
        rounds += 1
    dt = (time.perf_counter() - t0) / rounds
    A = out.accept_len.cpu().numpy()[reqs]
    am = out.argmax.cpu().numpy()
    row_idx = np.concatenate([np.arange(case["row_off"][b], case["row_off"][b + 1]) for b in reqs])
    gap = ref["top2_gap"]
    near = (gap < 1e-2) & (gap > 0)
    differs = am[row_idx] != ref["argmax"]
    return {"value": sub["T"] / dt, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": "%d of %d requests (%d window rows, %d draft tokens) per oracle round, %d round(s) of %.2f s"
                      % (n_req, cfg.B, sub["R"], sub["T"], rounds, dt),
            "accept_len_equal": int(np.sum(A == ref["accept_len"])), "requests_compared": len(reqs),
            "rows_compared": int(row_idx.size), "near_tie_rows": int(near.sum()),
            "argmax_differs_outside_near_ties": int((differs & ~near).sum()),
            "near_tie_head_probs": int((np.abs(ref["head_prob"] - cfg.tau) < 2e-3).sum())}


def measure(cfg, w, wdev, args, rank, world, local_rank, ranks, with_baseline, baseline_repeat):
    """All timings of one workload on this rank's GPU; rank 0 gets the record (the others None)."""
    import torch
    from gen import cases

    dev = "cuda:%d" % local_rank
    case = cases.make_case(cfg, lambda wb, h: cases.library_ref_argmax(wb, h, device=dev), weights=w)
    d = cases.to_device(case, dev, weights_dev=wdev)
    v = cases.make_verifier(d)
    T, R = case["T"], case["R"]
    P = T if case["sel_pos"] is None else int(case["sel_pos"].shape[0])
    out = cases.run(v, d, extras=True)
    torch.cuda.synchronize()
    if v.device_error() != 0:
        raise SystemExit("device reported a pipeline time-out")
    plan = v.plan(R, P)
    one_launch = P > 0 and v.plan_kernels(R, P) == 3     # LM-head and decision-head CTAs share a launch
    plan["kernels_per_round"] = v.plan_kernels(R, P)

    def barrier():
        torch.cuda.synchronize()
        ranks.barrier()
        torch.cuda.synchronize()

    stream = torch.cuda.current_stream()
    steps = args.steps
    fast_out = cases.run(v, d, extras=False)
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def region(fn, n):
        """n calls of fn between two events on the launching stream, a barrier and a synchronise on both sides."""
        barrier()
        e0, e1 = ev(), ev()
        e0.record(stream)
        for _ in range(n):
            fn()
        e1.record(stream)
        barrier()
        return ranks.max(e0.elapsed_time(e1) / n)

    round_fn = lambda: cases.run(v, d, extras=False, out=fast_out)
    for _ in range(args.warmup):
        round_fn()
    est_ms = region(round_fn, min(steps, 5))
    # every region is exactly `steps` rounds; it is repeated so that the timed regions add up to args.min_seconds
    repeats = args.repeats if args.repeats > 0 else int(min(400, max(3, np.ceil(args.min_seconds * 1e3 / (steps * est_ms)))))

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    # ---- (1) device-resident inputs: `repeats` regions of `steps` back-to-back rounds
    n0 = v.launch_count()
    regions = [region(round_fn, steps) for _ in range(repeats)]
    launches = (v.launch_count() - n0) // repeats
    ms_step = float(statistics.median(regions))
    # ---- (1b) the same number of rounds in ONE region: no idle gaps, the clocks the power cap allows in steady state
    sustained_ms = region(round_fn, steps * repeats)

    # ---- (2) the same rounds with the library's per-kernel events switched on (roofline of the LM head)
    prof_steps = int(min(steps * repeats, 1000))
    v.profile_enable(prof_steps)
    for _ in range(prof_steps):
        round_fn()
    torch.cuda.synchronize()
    stage_ms = [v.profile_read(s, prof_steps) for s in range(4)]
    v.profile_enable(0)
    lm_ms = ranks.max(float(np.mean(stage_ms[1])))
    stage_mean = [float(np.mean(s)) if s else 0.0 for s in stage_ms]

    # ---- (3) end to end through the host-buffer entry point: H2D + round + D2H + sync per step
    pin = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    hc = {k: pin(case[k]) for k in ("target_hidden", "draft_tokens", "draft_hidden", "csi", "sel_off", "sel_pos",
                                    "draft_q", "uniforms")}
    hk = pin(case["k_off"]) if cfg.K_hi > 0 else None
    hkw = dict(B=cfg.B, K=cfg.K if cfg.K_hi == 0 else 0, k_off=hk, T=T, sel_off=hc["sel_off"],
               sel_pos=hc["sel_pos"], draft_q=hc["draft_q"], uniforms=hc["uniforms"], extras=False)
    # the serving-loop form of the call: the pinned buffers are bound once, every step is one wisv_verify_host on them
    host_call = v.bind_host(hc["target_hidden"], hc["draft_tokens"], hc["draft_hidden"], hc["csi"], **hkw)
    host_out = host_call()
    for _ in range(min(args.warmup, 10)):
        host_call()
    e2e_repeats = max(3, min(repeats, int(np.ceil(0.5 * args.min_seconds * 1e3 / (steps * est_ms)))))
    e2e_regions = [region(host_call, steps) for _ in range(e2e_repeats)]
    e2e_ms = float(statistics.median(e2e_regions))
    h2d = sum(int(t.numel() * t.element_size()) for t in list(hc.values()) + [hk] if t is not None)
    d2h = 2 * 4 * cfg.B
    same = bool(torch.equal(host_out.accept_len, fast_out.accept_len.cpu()))
    # ---- (3b) the same call with the hidden states as the uplink delivers them (Section IV-A: b_h = 16 bits per
    # element): the drafter's as fp16, the target's as bf16; half the bytes cross PCIe
    hc16 = dict(hc)
    hc16["target_hidden"] = hc["target_hidden"].to(torch.bfloat16).pin_memory()
    hc16["draft_hidden"] = hc["draft_hidden"].to(torch.float16).pin_memory()
    host_call16 = v.bind_host(hc16["target_hidden"], hc16["draft_tokens"], hc16["draft_hidden"], hc16["csi"], **hkw)
    for _ in range(min(args.warmup, 10) + 1):
        host_call16()
    e2e16_regions = [region(host_call16, steps) for _ in range(e2e_repeats)]
    e2e16_ms = float(statistics.median(e2e16_regions))
    h2d16 = sum(int(t.numel() * t.element_size()) for t in list(hc16.values()) + [hk] if t is not None)
    clocks = sampler.stop() if rank == 0 else None

    rec = None
    if rank == 0:
        peaks, peak_kind = load_peaks()
        w_bytes = cfg.V * cfg.H * 2
        flops = 2.0 * R * cfg.H * cfg.V
        if one_launch:
            # the timed kernel also streams the bf16 block of W1 and evaluates the head on P positions
            w_bytes += cfg.d_J * (cfg.H_d + cfg.H) * 2
            flops += 2.0 * P * cfg.d_J * (cfg.H_d + cfg.H)
        hbm_bound = R < 256
        if hbm_bound:
            achieved = w_bytes / (lm_ms * 1e-3) / 1e9
            peak = float(peaks["hbm_gbs"])
            # the measured peak is a copy (read + write); a read-only stream can exceed it, so the fraction of the
            # data-sheet bandwidth is printed beside it
            roof = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "frac_nominal": achieved / NOMINAL_PEAKS["hbm_gbs"], "nominal_peak": NOMINAL_PEAKS["hbm_gbs"],
                    "traffic": captured_traffic(cfg.name)}
        else:
            achieved = flops / (lm_ms * 1e-3) / 1e12
            peak = float(peaks["bf16_tflops"])
            sus = float(peaks.get("bf16_tflops_sustained", peak))
            roof = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "frac_sustained": achieved / sus, "sustained_peak": sus,
                    "frac_nominal": achieved / NOMINAL_PEAKS["bf16_tflops"], "nominal_peak": NOMINAL_PEAKS["bf16_tflops"],
                    "traffic": captured_traffic(cfg.name)}
        kernel_name = lm_kernel_name(R, one_launch)
        roof.update({"kernel": kernel_name, "kernel_ms": lm_ms, "peak_source": peak_kind,
                     "algorithmic_bytes": w_bytes, "algorithmic_flops": flops,
                     "stage_ms": {"pack": stage_mean[0], "lm_head": stage_mean[1], "decision_head": stage_mean[2],
                                  "merge_scan": stage_mean[3]}})
        mhz = clocks.get("sm_mhz") if clocks else None
        dec = decision_stats(case, out, cfg)
        rec = {"value": aggregate(world, T, ms_step), "ms_per_step": ms_step, "steps": steps, "repeats": repeats,
               "ms_per_step_regions": region_stats(regions),
               "sustained": {"ms_per_step": sustained_ms, "rounds": steps * repeats,
                             "value": aggregate(world, T, sustained_ms)},
               "kcycles_per_step": (ms_step * mhz) if mhz else None,
               "config": config_block(cfg, case, {"parallelism": "requests sharded, 1 batch per GPU", "plan": plan}),
               "clocks": clocks, "gpu_launches": int(launches),
               "e2e": {"value": aggregate(world, T, e2e_ms), "unit": UNIT, "h2d_bytes_per_step": h2d,
                       "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": steps, "repeats": e2e_repeats,
                       "ms_per_step_regions": region_stats(e2e_regions), "matches_device_path": same,
                       "hidden_dtype": "f32",
                       "sixteen_bit_hidden": {"value": aggregate(world, T, e2e16_ms), "unit": UNIT,
                                              "ms_per_step": e2e16_ms, "h2d_bytes_per_step": h2d16,
                                              "d2h_bytes_per_step": d2h, "hidden_dtype": "target bf16, draft f16",
                                              "ms_per_step_regions": region_stats(e2e16_regions)}},
               "roofline": roof,
               "accepted_tokens_per_s": world * dec["accepted_tokens"] / (ms_step * 1e-3),
               "decisions": dec}
        if with_baseline:
            rec["cpu_baseline"] = oracle_check(case, out, cfg, args.oracle_rows if baseline_repeat else args.leg_oracle_rows,
                                               args.oracle_seconds, baseline_repeat)
    v.close()
    del d, v, out, fast_out
    torch.cuda.empty_cache()
    return rec


def lm_kernel_name(R, one_launch):
    # which LM-head kernel the library's plan uses: single CTAs up to 128 window rows, CTA pairs above
    on_pairs = R > 128
    if one_launch:
        return ("lmhead_pair_kernel (CTA pairs + decision-head clusters)" if on_pairs
                else "round_small_kernel (LM-head CTAs + decision-head CTAs)")
    return "lmhead_pair_kernel (CTA pairs)" if on_pairs else "gemm_rowreduce_kernel<LM head>"


def run_ours(args, rank, world, local_rank):
    import torch

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verifier has no CPU path")
    if local_rank == 0:
        from paper_2604_17701_b200 import build as cuda_build
        cuda_build.build()          # compiles the in-tree library only if it is missing or stale
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    ranks = Ranks(world, "nccl", dev)
    ranks.barrier()                 # the other ranks load the library only after rank 0 has it in place

    cfg = workload_config(args.workload, rank)
    legs = [n for n in args.legs if n != cfg.name and same_model(gen.config(n), cfg)]
    w, shm_path = shared_weights(cfg, rank, ranks)
    wdev = device_weights(w, dev)                       # one upload of the model for the headline and every leg
    try:
        head = measure(cfg, w, wdev, args, rank, world, local_rank, ranks, world == 1 and not args.no_cpu_baseline, True)
        leg_recs = {}
        for name in legs:
            lcfg = workload_config(name, rank)
            largs = argparse.Namespace(**vars(args))
            rec = measure(lcfg, w, wdev, largs, rank, world, local_rank, ranks,
                          world == 1 and not args.no_cpu_baseline, False)
            if rec is not None:
                rec.update({"metric": METRIC, "unit": UNIT, "dtype": "bf16"})
                leg_recs[name] = rec
    finally:
        if shm_path:
            try:
                os.unlink(shm_path)
            except OSError:
                pass
    if rank == 0:
        line = {"metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
        line.update({k: v for k, v in head.items() if k not in ("value", "ms_per_step", "steps")})
        # the accepted-token rate of Table I's "throughput" column needs rounds that accept something: one request at
        # B = 1 may reject at position 0, so the job-level figures average over the headline batch and the legs
        allrecs = [head] + list(leg_recs.values())
        line["mean_accept_len"] = float(np.mean([r["decisions"]["mean_accept_len"] for r in allrecs]))
        line["accepted_tokens_per_s_by_workload"] = {r["config"]["workload"]: r["accepted_tokens_per_s"] for r in allrecs}
        if leg_recs:
            line["legs"] = leg_recs
        print(json.dumps(line), flush=True)
    ranks.close()


def same_model(a, b):
    return (a.H, a.V, a.H_d, a.d_c, a.d_J, a.weight_seed) == (b.H, b.V, b.H_d, b.d_c, b.d_J, b.weight_seed) and a.weight_seed >= 0


def shard_bounds(V, world):
    """Vocabulary rows [lo, hi) of every rank: equal slices rounded to 16 rows."""
    per = -(-V // world)
    per = -(-per // 16) * 16
    return [(min(V, r * per), min(V, (r + 1) * per)) for r in range(world)]


def run_sharded(args, rank, world, local_rank):
    """The same batch on every GPU, the LM head split by vocabulary: shard rows -> all-gather -> merge (strong scaling)."""
    import torch
    from gen import cases

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the verifier has no CPU path")
    if local_rank == 0:
        from paper_2604_17701_b200 import build as cuda_build
        cuda_build.build()
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    ranks = Ranks(world, "nccl", dev)
    ranks.barrier()
    cfg = workload_config(args.workload)                   # one batch, seen by every rank
    case = cases.make_case(cfg, lambda w, h: cases.library_ref_argmax(w, h, device=dev))
    d = cases.to_device(case, dev)
    lo, hi = shard_bounds(cfg.V, world)[rank]
    if hi <= lo:
        raise SystemExit("more GPUs than 16-row slices of the vocabulary")
    v = cases.make_verifier(d, vocab_slice=(lo, hi))
    T, R = case["T"], case["R"]
    geo = dict(B=cfg.B, K=cfg.K if cfg.K_hi == 0 else 0, k_off=d["k_off_dev"], T=T)
    part = torch.empty((R, 4), dtype=torch.float32, device=dev)
    gathered = torch.empty((world, R, 4), dtype=torch.float32, device=dev)
    res = None

    def step():
        nonlocal res
        v.shard_rows(d["target_hidden"], d["draft_tokens"], out=part, **geo)
        ranks.all_gather(gathered, part)                            # R * 16 bytes per GPU over NVLink
        res = v.verify_gathered(gathered, d["target_hidden"], d["draft_tokens"], d["draft_hidden"], d["csi"],
                                sel_off=d["sel_off"], sel_pos=d["sel_pos"], draft_q=d["draft_q"],
                                uniforms=d["uniforms"], out=res, **geo)

    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize(); ranks.barrier(); torch.cuda.synchronize()
    n0 = v.launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    torch.cuda.synchronize(); ranks.barrier(); torch.cuda.synchronize()
    ms_step = ranks.max(e0.elapsed_time(e1) / args.steps)
    launches = v.launch_count() - n0
    # end to end: inputs from pinned host memory every step, accepted lengths read back
    pin = lambda t: None if t is None else t.cpu().pin_memory()
    host = {k: pin(d[k]) for k in ("target_hidden", "draft_tokens", "draft_hidden", "csi")}
    e2e_steps = max(3, min(args.steps, 200))
    back = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    torch.cuda.synchronize(); ranks.barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        for k, t in host.items():
            d[k].copy_(t, non_blocking=True)
        step()
        back.copy_(res.accept_len, non_blocking=True)
        torch.cuda.synchronize()
    e1.record(stream)
    torch.cuda.synchronize(); ranks.barrier()
    e2e_ms = ranks.max(e0.elapsed_time(e1) / e2e_steps)
    h2d = sum(int(t.numel() * t.element_size()) for t in host.values())
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0:
        peaks, peak_kind = load_peaks()
        shard_bytes = (hi - lo) * cfg.H * 2
        line = {"metric": METRIC, "value": T / (ms_step * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "strong",
                "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": config_block(cfg, case, {"parallelism": "LM head sharded by vocabulary over %d GPU(s), "
                                                                  "row partials all-gathered" % world,
                                                   "vocab_rows_per_gpu": hi - lo}),
                "clocks": clocks, "gpu_launches": int(launches),
                "e2e": {"value": T / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                        "d2h_bytes_per_step": 4 * cfg.B, "ms_per_step": e2e_ms, "steps": e2e_steps},
                # no per-kernel events in this mode: the shard's weight bytes over the WHOLE step (shard kernel,
                # all-gather, merge/scan), a lower bound on what the LM-head kernel alone achieves
                "roofline": {"bound": "hbm", "achieved": shard_bytes / (ms_step * 1e-3) / 1e9,
                             "peak": float(peaks["hbm_gbs"]), "unit": "GB/s",
                             "frac": shard_bytes / (ms_step * 1e-3) / 1e9 / float(peaks["hbm_gbs"]),
                             "traffic": None, "peak_source": peak_kind, "algorithmic_bytes": shard_bytes,
                             "kernel": "whole step (LM-head shard + all-gather + merge/scan)",
                             "note": "whole-step floor per GPU = shard bytes / peak = %.1f us" %
                                     (shard_bytes / float(peaks["hbm_gbs"]) / 1e3)},
                "mean_accept_len": float(res.accept_len.float().mean().item())}
        print(json.dumps(line), flush=True)
    v.close()
    ranks.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b_b1", choices=sorted(gen.CONFIGS))
    ap.add_argument("--shard", default="requests", choices=["requests", "vocab"],
                    help="multi-GPU split: independent batches per GPU (default), or one batch with the LM head "
                         "sharded by vocabulary")
    ap.add_argument("--legs", default=None,
                    help="comma-separated workloads of the same model measured after the headline one and printed under "
                         "'legs' (default at 1 GPU with the default workload: %s; 'none' switches them off)" % ",".join(DEFAULT_LEGS))
    ap.add_argument("--repeats", type=int, default=0,
                    help="timed regions of --steps rounds each (0: as many as add up to --min-seconds, at least 3)")
    ap.add_argument("--min-seconds", type=float, default=0.6,
                    help="the timed regions of a workload add up to about this much device time")
    ap.add_argument("--leg-oracle-rows", type=int, default=96,
                    help="window rows the oracle checks per leg (one round)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--oracle-seconds", type=float, default=10.0,
                    help="CPU-baseline leg: repeat the oracle round until this much time has passed")
    ap.add_argument("--oracle-rows", type=int, default=None,
                    help="window rows of oracle work per baseline round (bounds its run time)")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1 and world != args.gpus:
        raise SystemExit("--gpus must equal WORLD_SIZE under torchrun")
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        args.oracle_rows = 64 if args.oracle_rows is None else args.oracle_rows
        run_reference(args, rank, world)
    else:
        args.steps = 20 if args.steps is None else args.steps
        args.warmup = 5 if args.warmup is None else args.warmup
        args.warmup = max(3, args.warmup)
        args.oracle_rows = 800 if args.oracle_rows is None else args.oracle_rows
        if args.legs is None:
            args.legs = list(DEFAULT_LEGS) if (world == 1 and args.workload == "8b_b1" and args.shard == "requests") else []
        else:
            args.legs = [n for n in args.legs.split(",") if n and n != "none"]
            for n in args.legs:
                if n not in gen.CONFIGS:
                    raise SystemExit("unknown leg workload %r" % n)
        if args.shard == "vocab":
            run_sharded(args, rank, world, local_rank)
        else:
            run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
