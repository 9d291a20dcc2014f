#!/usr/bin/env python
"""Benchmark of the fused compression round (tri_compress) on synthetic Qwen3-shaped caches.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole hot path (phasor fold, scoring, z-score/max, top-B select, gather
compaction) over every (sequence, layer, KV head) unit of the workload.  Prints ONE JSON line.

* value       keys scored+selected+compacted per second on the headline workload (the 131,072-token
              sequence unless --workload says otherwise), inputs resident in HBM, CUDA events around exactly
              K steps, max over ranks (N > 1: independent replicas, one per GPU, "weak" scaling).
* sustained   the same workload run back to back for about one second (the power-capped regime), with the
              clock samples of that second.
* workloads   at N = 1 and without --workload: the other benchmark configurations (steady-state batch,
              32K one-shot, a 16-layer slab of the ragged paged batch) timed the same way, each with its
              achieved fraction of the HBM roofline.
* e2e         the headline metric through tri_compress_host: pinned host K/V in, compacted K/V out, copies
              inside the timed region.
* roofline    the scoring kernel (it streams the whole key cache): algorithmic bytes / its mean launch
              time, measured with CUDA events recorded by the library around its launches in a second
              pass of K steps.
* cpu_baseline  the float64 oracle, as it stands, on a bounded sample of units of the same workload.

--impl reference times that oracle alone (rank 0 only), one sampled unit per step.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "tri_compress keys scored+selected+compacted per sec"
UNIT = "keys/s"
DEFAULT_WORKLOAD = "qwen3_8b_long_128k"
# the other configurations a default run also times: (workload, layers; 0 = all)
OTHER_WORKLOADS = (("qwen3_8b_steady_b64", 0), ("qwen3_8b_oneshot_32k", 0), ("qwen3_32b_ragged_paged", 16))
NOMINAL_HBM_GBS = 8000.0


# DRAM traffic of the scoring kernel from its ncu capture (dram__bytes_read.sum + dram__bytes_write.sum of one launch of
# k_score_tma<1,0> on 1,048,576 keys: 268,527,872 B + 14,151,424 B), valid only for the kernel source it was taken on.
SCORE_TRAFFIC = {"bytes_per_key": (268527872 + 14151424) / 1048576,
                 "sources": ["paper_2604_04921_b200/csrc/tri_score_tma.cuh", "paper_2604_04921_b200/csrc/tri_score.cuh",
                             "paper_2604_04921_b200/csrc/tri_common.cuh"],
                 "sha256": "593d3dd118fbf9bc7c8d32a690de9d7e27d4efda005560991a4a4e1b577abc17"}


def score_traffic_per_launch(keys):
    """ncu traffic scaled to a launch of `keys` keys (it grows in proportion), or None if the kernel's
    source has changed since the counters were taken."""
    import hashlib
    h = hashlib.sha256()
    for rel in SCORE_TRAFFIC["sources"]:
        with open(os.path.join(ROOT, rel), "rb") as f:
            h.update(f.read())
    return SCORE_TRAFFIC["bytes_per_key"] * keys if h.hexdigest() == SCORE_TRAFFIC["sha256"] else None


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, an earlier measurement on B200)"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi for the life of the run; a timed region asks for
    the samples that fell between its mark() and its summary()."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        """Starts nvidia-smi and waits for its first sample: its start-up can stall the GPU for seconds and
        must not fall into a timed region."""
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "200"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
            t0 = time.time()
            while not self.rows and time.time() - t0 < 30.0 and self.proc.poll() is None:
                time.sleep(0.05)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def mark(self):
        """Index of the next sample (call right before a timed region)."""
        return len(self.rows)

    def summary(self, first: int):
        """Median SM clock and active throttle reasons of the samples taken since mark() returned `first`."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.06)
        last = len(self.rows)
        # a timed region shorter than the sampling period holds no sample: fall back to the whole run so far
        window = "timed region" if last > first else "whole run so far (timed region shorter than one sample)"
        rows = self.rows[first:last] if last > first else self.rows[:last]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except Exception:
                continue
            for nm, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "window": window, "reasons": sorted(reasons)}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()


def algorithmic_bytes(seq_lens, units_per_seq, budget, row_bytes=256):
    """256 N (stream K) + 1036 min(B, N) (re-read kept K, read kept V, write both, idx + positions); rows of
    row_bytes bytes in general: row_bytes N + (4 row_bytes + 12) min(B, N)."""
    tot = 0
    for n in seq_lens:
        tot += units_per_seq * (row_bytes * n + (4 * row_bytes + 12) * min(budget, n))
    return tot


def workload_config(spec, L, world=1):
    """The `config` object of the JSON line; both arms (the CUDA path and --impl reference) print the same one."""
    S, H = spec.n_seqs, spec.n_kv_heads
    return {"workload": spec.name + (f"[first {L} layers]" if L != spec.n_layers else ""),
            "units": L * S * H, "layers": L, "kv_heads": H, "group_size": spec.group_size, "seqs": S,
            "keys_per_unit": spec.n_keys if spec.kind != "ragged_paged" else f"{spec.n_keys_min}..{spec.n_keys}",
            "budget": spec.budget, "storage_dtype": "bf16", "accumulate_dtype": "f32", "paged": spec.kind == "ragged_paged",
            "compaction": "in place into the sequence's pages, pool restored between steps outside the timed region"
            if spec.kind == "ragged_paged" else "out of place",
            "l2": "inputs larger than L2 (GB of K+V per step in hbm.kv_bytes)",
            "parallelism": "replicas" if world > 1 else "single GPU"}


def oracle_sample(spec, units, budget):
    """Time the CPU oracle on the given (layer, seq, head) units.  Returns (keys, seconds)."""
    import oracle
    from paper_2604_04921_b200 import workloads as W
    keys, secs, cache = 0, 0.0, {}
    for (l, s, h) in units:
        if l not in cache:
            cache.clear()
            cache[l] = W.make_workload(spec, "cpu", layer0=l, n_layers=1)
        w = cache[l]
        kk, vv, pos = w.unit_rows(0, s, h)
        G = spec.group_size
        bits = W.bf16_bits(kk)
        qc = w.q_center[0, h * G:(h + 1) * G].double().numpy()
        qn = w.q_mean_norm[0, h * G:(h + 1) * G].double().numpy()
        t0 = time.perf_counter()
        raw, sfin, idx = oracle.unit_bf16(bits, pos.numpy(), int(w.cur_pos[s]), qc, qn, budget, theta=spec.theta)
        oracle.compact(W.bf16_bits(kk), idx)
        oracle.compact(W.bf16_bits(vv), idx)
        secs += time.perf_counter() - t0
        keys += kk.shape[0]
    return keys, secs


def sample_units(spec, count):
    """Deterministic spread of units: first/last layer and head first, then striding through."""
    L, S, H = spec.n_layers, spec.n_seqs, spec.n_kv_heads
    out = [(0, 0, 0), (L - 1, S - 1, H - 1)]
    i = 1
    while len(out) < count:
        u = (i * 7919) % (L * S * H)
        out.append((u // (S * H), (u // H) % S, u % H))
        i += 1
    return out[:count]


def max_over_ranks(ms, dist, device):
    """The slowest rank's time: MAX all-reduce over the process group (identity without one)."""
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world, keys_per_rank_step, ms_step):
    """Replicas: every rank processes the same number of keys per step; the job's rate is their sum
    over the slowest rank's step time."""
    return world * keys_per_rank_step / (ms_step * 1e-3)


def run_reference(args, spec):
    """--impl reference: the oracle as it stands, one sampled unit per step, on the host cores."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    if args.steps <= 0:
        args.steps = 4
    oracle.build()
    L = args.layers if args.layers > 0 else spec.n_layers
    units = sample_units(spec.scaled(n_layers=L), 1 + args.steps)
    oracle_sample(spec, units[:1], spec.budget)                      # warm-up: page in, build
    keys, secs = oracle_sample(spec, units[1:1 + args.steps], spec.budget)
    val = keys / secs
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * secs / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(spec, L),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": f"each step = one unit of the workload, {args.steps} units ({keys} keys) out of "
                                       f"{L * spec.n_seqs * spec.n_kv_heads}; one untimed warm-up unit"},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_calibration(args):
    """--calibration: the statistics pass that feeds the round (E[q_f], E|q_f|, R_f of one layer's query heads
    from bf16 pre-RoPE queries), on a Qwen3-8B-shaped layer: 32 heads x 262,144 tokens (the calibration sets of
    the paper's sensitivity study hold 50k to 960k tokens).  One step = one pass over the layer's queries."""
    import torch
    from paper_2604_04921_b200 import binding as tb
    from paper_2604_04921_b200 import workloads as W
    torch.cuda.set_device(0)
    tb.lib()
    sp = W.SPECS["qwen3_8b_oneshot_32k"]
    T, Hq = (args.tokens if args.tokens > 0 else 262144), sp.n_kv_heads * sp.group_size
    q = W.make_queries(sp, 0, T, "cuda", dtype=torch.bfloat16)
    cal = tb.Calibrator(Hq)
    for _ in range(max(3, args.warmup)):
        cal.add(q)
    torch.cuda.synchronize()
    steps = args.steps if args.steps > 0 else 1000
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(steps):
        cal.add(q)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    peak, peak_src = measured_peaks()
    nbytes = q.numel() * 2
    line = {"metric": "tri_calib_accumulate query rows (token x head) per sec", "value": T * Hq / (ms * 1e-3), "unit": "rows/s",
            "n_gpus": 1, "steps": steps, "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": "calibration qwen3_8b layer", "tokens": T, "heads": Hq, "storage_dtype": "bf16",
                       "l2": f"inputs larger than L2: {nbytes / 1e9:.2f} GB read per step"},
            "roofline": {"kernel": "k_calib_tma (+ k_calib_merge)", "bound": "hbm", "achieved": nbytes / (ms * 1e-3) / 1e9,
                         "peak": peak, "unit": "GB/s", "frac": nbytes / (ms * 1e-3) / 1e9 / peak, "traffic": None,
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": nbytes},
            "gpu_launches": 2 * steps}
    if not args.no_cpu_baseline:
        import oracle
        oracle.build()
        qs = q[:16384, :4].double().cpu().numpy()
        t0 = time.perf_counter()
        for h in range(4):
            oracle.calibrate(qs[:, h])
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 16384 * 4 / dt, "unit": "rows/s", "cores": 1, "kind": "oracle",
                                "sample": "16,384 tokens x 4 heads"}
    print(json.dumps(line), flush=True)


class Round:
    """One workload resident on the device with everything a timed tri_compress step needs."""

    def __init__(self, spec, L, dev, pre_rope=False, e4m3=False):
        import torch
        from paper_2604_04921_b200 import binding as tb
        from paper_2604_04921_b200 import workloads as W
        self.spec, self.L, self.dev = spec, L, dev
        self.w = w = W.make_workload(spec, dev, layer0=0, n_layers=L)
        self.row_bytes = 256
        if e4m3:
            # the same rows rounded to e4m3 (k_kind 3): 128-byte K and V rows
            w.k, w.v = w.k.float().to(torch.float8_e4m3fn), w.v.float().to(torch.float8_e4m3fn)
            self.row_bytes = 128
        S, H, G, B = spec.n_seqs, spec.n_kv_heads, spec.group_size, spec.budget
        self.ctx = tb.TriContext(L, H, G, w.q_center, w.q_mean_norm, rope_theta=spec.theta)
        # pre_rope: the same bf16 rows read as pre-RoPE vectors (k_kind 2): the kernels' work does not depend on the values
        self.src = tb.CacheView(w.k, w.v, seq_lens=w.seq_lens, positions=w.positions, page_table=w.page_table, pre_rope=pre_rope)
        self.n_max = self.src.c_view().n_max
        self.U = L * S * H
        if w.paged:
            # compacted rows are written back into the sequence's own pages (in place)
            self.dst = tb.CacheView(w.k, w.v, page_table=w.page_table, n_max=self.n_max, pre_rope=pre_rope)
            self.k2 = self.v2 = self.p2 = None
        else:
            self.k2 = torch.empty(L, S, H, B, 128, dtype=w.k.dtype, device=dev)
            self.v2 = torch.empty_like(self.k2)
            self.p2 = torch.empty(L, S, H, B, dtype=torch.int32, device=dev)
            self.dst = tb.CacheView(self.k2, self.v2, positions=self.p2, pre_rope=pre_rope)
        self.ws = self.ctx.workspace(S, self.n_max, B, dev)
        self.kept_cnt = torch.zeros(self.U, dtype=torch.int32, device=dev)
        self.lens = w.seq_lens.tolist()
        self.keys_per_step = sum(self.lens) * L * H
        self.abytes = algorithmic_bytes(self.lens, L * H, B, self.row_bytes)
        self.launches_per_step = self.ctx.compress_launches(self.src, S, self.dst)
        # An in-place round changes its own input (the kept rows move to the front of each sequence's pages), and
        # a second round on that state would find nearly every kept row already in place.  So for the paged
        # workload every step starts from the pristine pool: the pages a round overwrites are put back from a copy
        # between steps, outside the timed region, and each step is timed on its own.
        self.restore = None
        if w.paged:
            ps = spec.page_size
            keep_pages = (B + ps - 1) // ps
            pages = torch.cat([w.page_table[s, :min(keep_pages, (self.lens[s] + ps - 1) // ps)] for s in range(S)]).long()
            k_bak, v_bak = w.k[:, pages].clone(), w.v[:, pages].clone()

            def restore():
                w.k[:, pages] = k_bak
                w.v[:, pages] = v_bak
            self.restore = restore

    def step(self):
        self.ctx.compress(self.src, self.w.cur_pos, self.spec.budget, self.dst, self.ws, kept_cnt=self.kept_cnt)

    def timed_steps(self, n):
        """n steps; returns their total device time in ms (this rank)."""
        import torch
        if self.restore is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n):
                self.step()
            e1.record()
            torch.cuda.synchronize()
            return e0.elapsed_time(e1)
        evs = []
        for _ in range(n):
            self.restore()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            self.step()
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return sum(a.elapsed_time(b) for a, b in evs)

    def warm(self, n):
        for _ in range(n):
            if self.restore is not None:
                self.restore()
            self.step()

    def kernel_ms(self, steps):
        """Mean duration of each kernel kind per step: events recorded by the library around its launches."""
        self.ctx.profile_begin()
        per = {k: 0.0 for k in self.ctx.KERNELS}
        for _ in range(steps):
            if self.restore is not None:
                self.restore()
            self.step()
            for k, v in self.ctx.profile_read().items():
                per[k] += v / steps
        self.ctx.profile_end()
        return per

    def hbm(self, ms_step, peak):
        gbs = self.abytes / (ms_step * 1e-3) / 1e9
        return {"algorithmic_bytes_per_step": self.abytes, "kv_bytes": (self.w.k.numel() + self.w.v.numel()) * self.w.k.element_size(),
                "achieved_gbs": gbs, "frac_of_measured_copy_peak": gbs / peak, "frac_of_nominal_8tbs": gbs / NOMINAL_HBM_GBS}

    def close(self):
        self.ctx.close()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed steps; 0 = as many as fill about one second")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--workload", default=None, help=f"headline workload (default {DEFAULT_WORKLOAD}, plus the others)")
    ap.add_argument("--layers", type=int, default=0, help="only the first LAYERS layers (a slab); 0 = all")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", action="store_true", help="time the headline workload only")
    ap.add_argument("--e4m3", action="store_true", help="the workload's K and V rounded to e4m3 (k_kind 3: 128-byte rows, f16 tensor-core scoring)")
    ap.add_argument("--pre-rope", action="store_true", help="treat the bf16 keys as pre-RoPE vectors (k_kind 2: fp32 scoring with phasor tables)")
    ap.add_argument("--calibration", action="store_true", help="time the calibration-statistics pass instead of the round")
    ap.add_argument("--tokens", type=int, default=0, help="--calibration: tokens per pass (default 262,144)")
    args = ap.parse_args()
    if args.calibration:
        run_calibration(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "b200" else args.warmup

    from paper_2604_04921_b200 import workloads as W
    others = args.workload is None and args.layers == 0 and not args.no_others and not args.pre_rope and not args.e4m3
    spec = W.SPECS[args.workload or DEFAULT_WORKLOAD]
    if args.impl == "reference":
        run_reference(args, spec)
        return

    import torch
    from paper_2604_04921_b200 import binding as tb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the compression round has no CPU implementation")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    tb.lib()   # fails loudly if the CUDA library has not been built

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    peak, peak_src = measured_peaks()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()

    def second_of_steps(rd):
        """About one second of back-to-back steps (the power-capped regime) with its clock samples."""
        est = max_over_ranks(rd.timed_steps(3) / 3, dist, dev)
        barrier()
        n = int(min(3000, max(20, 1000.0 / est)))
        first = sampler.mark()
        ms = max_over_ranks(rd.timed_steps(n), dist, dev) / n
        barrier()
        return n, ms, (sampler.summary(first) if rank == 0 else None)

    L = args.layers if args.layers > 0 else spec.n_layers
    rd = Round(spec, L, dev, pre_rope=args.pre_rope, e4m3=args.e4m3)
    rd.warm(args.warmup)
    barrier()
    sustained = None
    if args.steps <= 0:
        args.steps, ms_step, clocks = second_of_steps(rd)
    else:
        first = sampler.mark()
        ms_step = max_over_ranks(rd.timed_steps(args.steps), dist, dev) / args.steps
        barrier()
        clocks = sampler.summary(first) if rank == 0 else None
        n, ms, ck = second_of_steps(rd)
        sustained = {"steps": n, "ms_per_step": ms, "value": whole_job_value(world, rd.keys_per_step, ms), "unit": UNIT,
                     "hbm": rd.hbm(ms, peak), "clocks": ck}

    per = rd.kernel_ms(min(args.steps, 50))
    score_bytes = rd.row_bytes * rd.keys_per_step
    score_gbs = score_bytes / (per["score"] * 1e-3) / 1e9
    cfg = workload_config(spec, L, world)
    if args.pre_rope:
        cfg["keys"] = "bf16 pre-RoPE (k_kind 2)"
    if args.e4m3:
        cfg["keys"] = "e4m3 post-RoPE keys and e4m3 values (k_kind 3), 128-byte rows"
        cfg["storage_dtype"] = "e4m3"
    line = {
        "metric": METRIC, "value": whole_job_value(world, rd.keys_per_step, ms_step), "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f16" if args.e4m3 else "bf16", "data": "synthetic",
        "config": cfg,
        "keys_per_step": rd.keys_per_step,
        "hbm": rd.hbm(ms_step, peak),
        "roofline": {"kernel": "k_score_tma<e4m3>" if args.e4m3 else "k_score_bf16_pre" if args.pre_rope else ("k_score_umma" if spec.group_size > 4 else "k_score_tma"), "bound": "hbm", "achieved": score_gbs, "peak": peak, "unit": "GB/s",
                     "frac": score_gbs / peak, "traffic": score_traffic_per_launch(rd.keys_per_step) if (spec.group_size <= 4 and not args.pre_rope and not args.e4m3) else None, "peak_source": peak_src,
                     "algorithmic_bytes_per_launch": score_bytes, "ms_per_launch": per["score"],
                     "note": "per step; a pipelined round issues the scoring as several launches over unit ranges, "
                             "their bytes and durations are summed"},
        "kernel_ms": per,
        "gpu_launches": rd.launches_per_step * args.steps,
        "clocks": clocks,
    }
    if sustained is not None:
        line["sustained"] = sustained

    # ---- end to end through tri_compress_host: pinned host buffers, copies inside the timed region ----
    w, S, B, U = rd.w, spec.n_seqs, spec.budget, rd.U
    if not args.no_e2e and not w.paged and not args.e4m3:
        e2e_steps = max(2, min(args.steps, 3 if rd.keys_per_step > 2e7 else 5))
        hk = torch.empty(w.k.shape, dtype=w.k.dtype, pin_memory=True).copy_(w.k)
        hv = torch.empty(w.v.shape, dtype=w.v.dtype, pin_memory=True).copy_(w.v)
        hpos = None if w.positions is None else torch.empty(w.positions.shape, dtype=torch.int32, pin_memory=True).copy_(w.positions)
        hlens = torch.empty(S, dtype=torch.int32, pin_memory=True).copy_(w.seq_lens)
        hcur = torch.empty(S, dtype=torch.int64, pin_memory=True).copy_(w.cur_pos)
        hk2 = torch.empty(rd.k2.shape, dtype=rd.k2.dtype, pin_memory=True)
        hv2 = torch.empty(rd.k2.shape, dtype=rd.k2.dtype, pin_memory=True)
        hp2 = torch.empty(rd.p2.shape, dtype=torch.int32, pin_memory=True)
        hcnt = torch.empty(U, dtype=torch.int32, pin_memory=True)
        dlens = torch.empty_like(w.seq_lens)
        dcur = torch.empty_like(w.cur_pos)
        src_h = tb.CacheView(hk, hv, seq_lens=hlens, positions=hpos)
        src_d = tb.CacheView(w.k, w.v, seq_lens=dlens, positions=w.positions)
        dst_h = tb.CacheView(hk2, hv2, positions=hp2)

        def step_host():
            rd.ctx.compress_host(src_h, src_d, hcur, dcur, B, dst_h, rd.dst, hcnt, rd.kept_cnt, rd.ws)

        step_host()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            step_host()
        e1.record()
        barrier()
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), dist, dev) / e2e_steps
        assert int(hcnt.min()) == min(B, min(rd.lens))
        # K is copied in full; of V and the positions only the kept rows cross the link (read by the gather
        # straight from the pinned host arrays)
        kept_rows = sum(min(B, n) for n in rd.lens) * L * spec.n_kv_heads
        if 2 * B <= rd.n_max:
            h2d = hk.numel() * 2 + kept_rows * 256 + (0 if hpos is None else kept_rows * 4) + S * 12
        else:       # most rows are kept: V and positions are staged in bulk like K
            h2d = (hk.numel() + hv.numel()) * 2 + (0 if hpos is None else hpos.numel() * 4) + S * 12
        d2h = (hk2.numel() + hv2.numel()) * 2 + hp2.numel() * 4 + U * 4
        line["e2e"] = {"value": whole_job_value(world, rd.keys_per_step, ms_e2e), "unit": UNIT, "ms_per_step": ms_e2e,
                       "steps": e2e_steps, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                       "call": "tri_compress_host (pinned host K/V/positions in, compacted K/V/positions/counts out; V and positions of kept rows read in place)"}
        del hk, hv, hk2, hv2, hpos, hp2, src_h, dst_h
    else:
        line["e2e"] = None

    # ---- the oracle on this machine's host cores, bounded sample (rank 0, N = 1 only) ----
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        if rd.restore is not None:
            rd.restore()
        G = spec.group_size
        units = sample_units(spec.scaled(n_layers=L), 512)
        keys = secs = 0.0
        used = 0
        for (l, s, h) in units:                      # rows come from the workload already in HBM
            kk, vv, pos = w.unit_rows(l, s, h)
            bits, vbits = W.bf16_bits(kk), W.bf16_bits(vv)
            qc = w.q_center[l, h * G:(h + 1) * G].double().numpy()
            qn = w.q_mean_norm[l, h * G:(h + 1) * G].double().numpy()
            t0 = time.perf_counter()
            _, _, idx = oracle.unit_bf16(bits, pos.numpy(), int(w.cur_pos[s]), qc, qn, B, theta=spec.theta)
            oracle.compact(bits, idx)
            oracle.compact(vbits, idx)
            secs += time.perf_counter() - t0
            keys += kk.shape[0]; used += 1
            if secs > 12.0:
                break
        line["cpu_baseline"] = {"value": keys / secs, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                                "sample": f"{used} of {U} units ({int(keys)} keys), oracle time {secs:.1f} s"}

    # ---- the other benchmark configurations, same method (N = 1, default run only) ----
    if others and world == 1:
        rd.close()
        del rd, w
        torch.cuda.empty_cache()
        entries = [{"workload": cfg["workload"], "steps": (sustained or {}).get("steps", args.steps),
                    "ms_per_step": (sustained or {}).get("ms_per_step", ms_step),
                    "value": (sustained or {}).get("value", line["value"]), "unit": UNIT,
                    "hbm": (sustained or {}).get("hbm", line["hbm"]), "kernel_ms": per,
                    "clocks": (sustained or {}).get("clocks", clocks), "burst_ms_per_step": ms_step, "burst_steps": args.steps}]
        for name, layers in OTHER_WORKLOADS:
            if name == spec.name:
                continue
            sp = W.SPECS[name]
            Lo = layers if layers > 0 else sp.n_layers
            r2 = Round(sp, Lo, dev)
            r2.warm(3)
            torch.cuda.synchronize()
            first = sampler.mark()
            burst = r2.timed_steps(20) / 20
            n, ms, ck = second_of_steps(r2)
            entries.append({"workload": workload_config(sp, Lo)["workload"], "steps": n, "ms_per_step": ms,
                            "value": r2.keys_per_step / (ms * 1e-3), "unit": UNIT, "hbm": r2.hbm(ms, peak),
                            "kernel_ms": r2.kernel_ms(min(n, 20)), "clocks": ck, "burst_ms_per_step": burst, "burst_steps": 20,
                            "units": r2.U, "keys_per_step": r2.keys_per_step})
            r2.close()
            del r2
            torch.cuda.empty_cache()
        line["workloads"] = entries

    if rank == 0:
        sampler.stop()
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
