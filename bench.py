#!/usr/bin/env python
"""Benchmark of the PQ-HSA decode-step attention operator on B200.

One "step" = one pqhsa_decode call (LUT build, ADC scan with fused per-list sums, top-k,
hybrid attention) over one batch of synthetic sequences whose index and paged KV cache are
resident in HBM.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c3_b8_r1] [--impl reference]

Under torchrun (N > 1) every rank runs the same workload on its own GPU with its own seed
(the operator shards over sequences with no exchange step): weak scaling, value = the sum
over ranks of algorithmic bytes / max-over-ranks step time.

Beside the contract keys the line carries: `roofline` (the scan kernel against the measured
copy bandwidth, its DRAM traffic from an ncu capture, per-stage times from
pqhsa_decode_events and the utilisation of the shared-memory pipe, which is what binds the
scan), `e2e` (pqhsa_decode_host: query from pinned host memory, output read back),
`cpu_baseline` (the float64 oracle on whole sequences for about 10 s), `variants` (the other
config-3 shapes), `dense_comparator` (the library's dense decode kernel on the same cache,
and the ideal time of one read of K and V), `graph_replay_us_per_step` and `index_update`
(index maintenance, amortised over the 256 steps between two calls).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

METRIC = ("decode-attention achieved HBM GB/s at 128K context "
          "(algorithmic bytes per step / device time per step; us/step = 1000*ms_per_step)")
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
L2_FLUSH_BYTES = 512 << 20
# DRAM traffic of ONE scan launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture of this repository's scan kernel, see the profile summaries), keyed by workload: the
# figure is reported only for the workload it was captured on.
SCAN_DRAM_TRAFFIC = {"c3_b8_r1": 336.1e6 + 111.0e6}


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


# ------------------------------------------------------------------ algorithmic bytes
def algorithmic_bytes(cfg, seq_lens, budget_ppm):
    """Bytes one step must move.  Per sequence and KV head:
    codes M + norm 4 + list id 2 per token; one score row per query head written once and
    read once (4+4 B per token per query head); k exact K and V rows of 2*d*2 B per query
    head plus 64 B for the two 32-byte sectors that return the token's score and list id;
    one centroid row and one value-mean row (4*d B each) per list; the codebooks once;
    the lookup table written and read once."""
    d, M, G, nc = cfg.head_dim, cfg.pq_m, cfg.group, cfg.pq_ncode
    cb = M if nc > 16 else M // 2          # bytes of codes per token (two 4-bit codes per byte)
    total = scan = select = attend = lut = 0
    for n in seq_lens:
        n_s = min(cfg.n_sink, n)
        n_r = max(n_s, n - cfg.n_local) - n_s                  # indexed region
        k = min(n_r, (n_r * budget_ppm + 999_999) // 1_000_000)
        if cfg.exact_set_multiple > 1:
            fixed = n - n_r
            m_ = cfg.exact_set_multiple
            k = min(n_r, (fixed + k + m_ - 1) // m_ * m_ - fixed)
        k += n - n_r                                           # rows attended exactly: T, S and L
        lut_b = cfg.n_list * 4 * d + M * nc * cfg.pq_dsub * 4 + G * M * nc * 4 + G * cfg.n_list * 4
        scan_b = n * (cb + 4 + 2) + G * n * 4 + G * M * nc * 4 + G * cfg.n_list * 4
        sel_b = G * n * 4 + G * k * 4
        att_b = G * k * (2 * d * 2 + 64) + cfg.n_list * 4 * d + G * d * 2 * 2
        lut += cfg.n_kv_heads * lut_b
        scan += cfg.n_kv_heads * scan_b
        select += cfg.n_kv_heads * sel_b
        attend += cfg.n_kv_heads * att_b
    total = lut + scan + select + attend
    return dict(total=total, lut=lut, scan=scan, select=select, attend=attend)


def dense_attention_bytes(cfg, seq_lens):
    return sum(cfg.n_kv_heads * n * 2 * cfg.head_dim * 2 for n in seq_lens)


# ------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.rows, self.proc, self.thread = [], None, None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.gpu_index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        def pump():
            for line in self.proc.stdout:
                self.rows.append([x.strip() for x in line.split(",")])
        self.thread = threading.Thread(target=pump, daemon=True)
        self.thread.start()

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, pw = [], [], set(), []
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1])); pw.append(float(r[2]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown",
                                "sw_power_cap"), r[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None,
                    sm_max_mhz=max(mx) if mx else None,
                    power_w_max=max(pw) if pw else None,
                    samples=len(sm), reasons=sorted(reasons))


# ------------------------------------------------------------------ oracle (CPU baseline / reference arm)
def oracle_arrays_seq0(inp, idx):
    """Float64 host copies of what the oracle needs for sequence 0 (index arrays and its own
    KV pages); see tests/helpers.py."""
    from helpers import oracle_arrays_for_sequence
    return oracle_arrays_for_sequence(inp, idx, 0)


def oracle_sample(inp, arrays, cfg, budget_ppm, n_heads):
    """Runs the float64 oracle, as it stands, on the one sequence `arrays` holds and its first
    n_heads query heads.  Returns (seconds, algorithmic bytes of that sample)."""
    from helpers import run_oracle
    t0 = time.perf_counter()
    run_oracle(inp, None, budget_ppm=budget_ppm, heads=list(range(n_heads)), batch_items=[0],
               arrays=arrays)
    dt = time.perf_counter() - t0
    n = int(arrays["seq_lens"][0])
    frac = n_heads / cfg.n_q_heads
    return dt, algorithmic_bytes(cfg, [n], budget_ppm)["total"] * frac


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        n = 1
    return n


# ------------------------------------------------------------------ main
def parse_workload(name):
    from paper_2609_33746_b200.workload import named_config
    return named_config(name)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="c3_b8_r1",
                    help="c3_b{1,8}_r{1,2} (128K, headline), c2, c4, c5_n{16..512}_b{1,32}")
    ap.add_argument("--impl", default="pqhsa", choices=["pqhsa", "reference"])
    ap.add_argument("--kmeans-iters", type=int, default=4,
                    help="Lloyd iterations of the synthetic index (timing does not depend on it)")
    ap.add_argument("--no-variants", action="store_true",
                    help="skip the extra c3 variants (B=1, 2%%) reported beside the headline")
    ap.add_argument("--oracle-heads", type=int, default=8,
                    help="query heads of sequence 0 one step of the reference arm runs")
    ap.add_argument("--oracle-seconds", type=float, default=10.0,
                    help="the CPU baseline adds whole sequences until it has run this long")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference" and rank != 0:
        return 0

    import torch
    import dataclasses
    from paper_2609_33746_b200.index_builder import build_index
    from paper_2609_33746_b200.workload import generate

    if args.impl == "reference":
        # The oracle arm needs sequence 0 only (same seeds, hence the same keys, values,
        # queries and index as sequence 0 of the CUDA arm's workload).
        cfg = parse_workload(args.workload)
        cfg = dataclasses.replace(cfg, batch=1, seq_lens=cfg.seq_lens[:1],
                                  kmeans_iters=args.kmeans_iters)
        dev = "cuda:0" if torch.cuda.is_available() else "cpu"
        inp = generate(cfg, device=dev)
        idx = build_index(inp)
        arrays = oracle_arrays_seq0(inp, idx)
        heads = max(1, min(args.oracle_heads, cfg.n_q_heads))
        for _ in range(min(args.warmup, 1)):
            oracle_sample(inp, arrays, cfg, cfg.budget_ppm, heads)
        times, nbytes = [], 0
        for _ in range(args.steps):
            dt, nbytes = oracle_sample(inp, arrays, cfg, cfg.budget_ppm, heads)
            times.append(dt)
        ms = 1000.0 * sum(times) / len(times)
        val = nbytes / (ms * 1e-3) / 1e9
        full = parse_workload(args.workload)
        sample = (f"each step = float64 numpy oracle on sequence 0, query heads 0..{heads - 1} of "
                  f"{cfg.n_q_heads} ({heads / cfg.n_q_heads / full.batch:.4f} of the workload's step)")
        line = dict(impl="reference", metric=METRIC, value=val, unit="GB/s", n_gpus=args.gpus,
                    steps=args.steps, warmup=args.warmup, ms_per_step=ms, higher_is_better=True,
                    scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                    config=dict(workload=full.name, batch=full.batch, context=full.max_seq_len,
                                budget_ppm=full.budget_ppm, sample=sample),
                    cpu_baseline=dict(value=val, unit="GB/s", cores=cpu_threads(), kind="oracle",
                                      sample=sample, host_cpus=os.cpu_count()),
                    e2e=dict(value=val, unit="GB/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
        print(json.dumps(line))
        return 0

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decode path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    dist = None
    if world > 1 and args.impl != "reference":
        import torch.distributed as dist_mod
        dist = dist_mod
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device(dev))

    cfg = parse_workload(args.workload)
    cfg = dataclasses.replace(cfg, kmeans_iters=args.kmeans_iters, seed=cfg.seed + 97 * rank)
    t_gen = time.perf_counter()
    inp = generate(cfg, device=dev)
    idx = build_index(inp)
    torch.cuda.synchronize()
    t_gen = time.perf_counter() - t_gen
    seq_lens = list(cfg.seq_lens)

    # ---------------------------------------------------------------- our arm
    from paper_2609_33746_b200 import pqhsa
    from paper_2609_33746_b200.runner import DecodeOp

    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def time_decode(op, steps, warmup, staged_events=False):
        """Per-step device times (ms) of pqhsa_decode with an L2 flush between steps.
        With staged_events, also per-stage times from pqhsa_decode_events."""
        for _ in range(warmup):
            flush.zero_()
            op.decode()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(5 if staged_events else 2)]
              for _ in range(steps)]
        if staged_events:
            for row in ev:
                for e in row:
                    e.record()
        barrier()
        t0 = time.perf_counter()
        for i in range(steps):
            flush.zero_()
            if staged_events:
                pqhsa.decode_events(op.params, op.q, op.index, op.kv, op.seq_lens, op.out, op.ws,
                                    ev[i])
            else:
                ev[i][0].record()
                op.decode()
                ev[i][1].record()
        barrier()
        wall = time.perf_counter() - t0
        if staged_events:
            stages = [[row[j].elapsed_time(row[j + 1]) for j in range(4)] for row in ev]
            return [sum(s) for s in stages], stages, wall
        return [a.elapsed_time(b) for a, b in ev], None, wall

    def reduce_max(x):
        if dist is None:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    def measure(op, cfg_v, ppm, steps, warmup, lens):
        times, _, _ = time_decode(op, steps, warmup)
        ms = reduce_max(sum(times) / len(times))
        ab = algorithmic_bytes(cfg_v, lens, ppm)
        gbs = world * ab["total"] / (ms * 1e-3) / 1e9
        srt = sorted(times)
        return dict(ms=ms, gbs=gbs, bytes=ab, p10=srt[len(srt) // 10], p50=srt[len(srt) // 2],
                    p90=srt[(9 * len(srt)) // 10])

    try:
        gpu_index = int(os.environ.get("CUDA_VISIBLE_DEVICES", "").split(",")[local_rank])
    except Exception:
        gpu_index = local_rank
    sampler = ClockSampler(gpu_index)
    op = DecodeOp(inp, idx, device=dev)
    op.decode()
    torch.cuda.synchronize()
    assert op.device_status() == pqhsa.OK

    sampler.start()
    time.sleep(0.3)                      # let nvidia-smi come up before the first timed step
    head = measure(op, cfg, cfg.budget_ppm, args.steps, args.warmup, seq_lens)
    launches = args.steps * pqhsa.decode_launch_count(op.params)

    # per-stage times of the same call, recorded by the library around its own stages
    _, stages, _ = time_decode(op, args.steps, 2, staged_events=True)
    stage_ms = [statistics.mean(s[j] for s in stages) for j in range(4)]
    peak, peak_src = measured_peak()
    scan_bytes = head["bytes"]["scan"]
    scan_gbs = scan_bytes / (stage_ms[1] * 1e-3) / 1e9
    scan_traffic = SCAN_DRAM_TRAFFIC.get(cfg.name)
    roofline = dict(bound="hbm", kernel="scan_kernel (ADC scan + fused per-list sums)",
                    achieved=scan_gbs, peak=peak, unit="GB/s", frac=scan_gbs / peak,
                    peak_source=peak_src, traffic=scan_traffic,
                    traffic_note="dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture "
                                 "of one scan launch on this workload (null: not captured on it)",
                    binding_unit="the SM's load/store data pipe (one wavefront per clock: 16 B of "
                                 "table reads per token, subspace and head group), not HBM",
                    algorithmic_bytes_per_launch=scan_bytes, avg_launch_ms=stage_ms[1],
                    stage_ms=dict(lut=stage_ms[0], scan=stage_ms[1], select=stage_ms[2],
                                  attend=stage_ms[3]),
                    whole_step_frac_of_peak=head["gbs"] / world / peak)
    # the unit that binds the scan: a lower bound on its time from the table reads alone
    # (M 16-byte reads per token and head group at 128 B per SM and clock), filled in below
    # with the sampled clock
    scan_tiles = cfg.n_kv_heads * ((cfg.group + 3) // 4) * sum((n + 31) // 32 for n in seq_lens)
    roofline["data_pipe"] = dict(
        table_wavefronts_per_tile=(cfg.pq_m if cfg.pq_ncode > 16 else cfg.pq_m) * 4,
        tiles_per_launch=scan_tiles)

    # the attend stage against the memory system's price for its gather: a probe that reads the
    # selected tokens' K and V rows (same addresses, through the block table) and computes
    # nothing, timed like a stage (after the L2 flush, whose dirty lines the kernel that follows
    # has to write back) and once more behind a read sweep that leaves L2 clean
    sel_idx = op.decode_buffer(pqhsa.BUF_SEL_IDX, torch.int32)
    sel_count = op.decode_buffer(pqhsa.BUF_SEL_COUNT, torch.int32)
    sink = torch.zeros(4, dtype=torch.int32, device=dev)
    sweep_src = torch.empty(256 << 20, dtype=torch.uint8, device=dev).zero_()

    def probe_us(after_flush):
        ts = []
        for _ in range(12):
            if after_flush:
                flush.zero_()
            else:
                flush.zero_()
                sweep_src.sum()                       # reads 256 MB: what L2 holds afterwards is clean
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            pqhsa.gather_probe(op.params, op.kv, sel_idx, sel_count, op.seq_lens, sink)
            b.record()
            torch.cuda.synchronize()
            ts.append(1000 * a.elapsed_time(b))
        return statistics.median(ts[2:])
    gather_bytes = int(sel_count.sum().item()) * 2 * cfg.head_dim * 2      # a K and a V row per selected token
    pu_dirty, pu_clean = probe_us(True), probe_us(False)
    roofline["attend_gather_probe"] = dict(
        what="pqhsa_gather_probe: the selected K/V rows read through the block table, nothing computed",
        bytes=gather_bytes, us_after_dirty_l2_flush=pu_dirty, us_after_clean_l2=pu_clean,
        gbs_after_dirty_l2_flush=gather_bytes / pu_dirty / 1e3, gbs_after_clean_l2=gather_bytes / pu_clean / 1e3,
        attend_stage_us=1000 * stage_ms[3])
    del sweep_src

    # end to end through the host-buffer entry point: q from pinned host memory, out back
    q_host = op.q.cpu().pin_memory()
    out_host = torch.empty_like(q_host).pin_memory()
    q_stage, out_stage = torch.empty_like(op.q), torch.empty_like(op.q)
    for _ in range(3):
        pqhsa.decode_host(op.params, q_host, q_stage, op.index, op.kv, op.seq_lens, out_stage,
                          out_host, op.ws)
    barrier()
    e2e_times = []
    for _ in range(args.steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        pqhsa.decode_host(op.params, q_host, q_stage, op.index, op.kv, op.seq_lens, out_stage,
                          out_host, op.ws)
        e2e_times.append(time.perf_counter() - t0)
    barrier()
    e2e_ms = reduce_max(1000.0 * sum(e2e_times) / len(e2e_times))
    qbytes = op.q.numel() * op.q.element_size()
    e2e = dict(value=world * head["bytes"]["total"] / (e2e_ms * 1e-3) / 1e9, unit="GB/s",
               ms_per_step=e2e_ms, h2d_bytes_per_step=qbytes, d2h_bytes_per_step=qbytes,
               note="pqhsa_decode_host: q from pinned host memory, output read back, stream "
                    "synchronised, host wall clock; index and paged KV cache stay resident in HBM")

    # the other c3 variants (same tensors: batch 1 = sequence 0, 2% = another budget)
    variants = {}
    if cfg.name.startswith("c3") and not args.no_variants:
        for vb, vp in ((1, 10000), (1, 20000), (8, 10000), (8, 20000)):
            if vb > cfg.batch or (vb == cfg.batch and vp == cfg.budget_ppm):
                continue
            cfg_v = dataclasses.replace(cfg, batch=vb, seq_lens=cfg.seq_lens[:vb], budget_ppm=vp)
            inp_v = dataclasses.replace(inp, cfg=cfg_v)
            op_v = DecodeOp(inp_v, idx, device=dev, budget_ppm=vp)
            r = measure(op_v, cfg_v, vp, args.steps, args.warmup, list(cfg_v.seq_lens))
            variants[f"c3_b{vb}_r{vp // 10000}"] = dict(
                us_per_step=1000 * r["ms"], us_p10=1000 * r["p10"], us_p90=1000 * r["p90"],
                achieved_gbs=r["gbs"] / world, pct_of_8TBps=100 * r["gbs"] / world / NOMINAL_HBM_GBS,
                algorithmic_mb=r["bytes"]["total"] / 1e6)
            del op_v
        # the same workload with the scan's tables held in fp16 (opt-in; not the mode the parity
        # tolerances of the scan are stated for): approximate scores with the exact top-k on them,
        # and the same plus the fp32 re-score of the threshold zone, which selects what fp32 tables select
        for tag, mode, note in (
                ("+fp16_tables", True, "opt-in table_precision = fp16: approximate scores, exact top-k "
                                       "on them; the headline runs with fp32 tables"),
                ("+fp16_tables_rescore", "rescore", "opt-in table_precision = fp16 + fp32 re-score of the "
                                                    "tokens within the rounding bound of the k-th score: "
                                                    "the selected set of the fp32 tables")):
            op_h = DecodeOp(inp, idx, device=dev, fp16_tables=mode)
            r = measure(op_h, cfg, cfg.budget_ppm, args.steps, args.warmup, seq_lens)
            variants[cfg.name + tag] = dict(
                us_per_step=1000 * r["ms"], us_p10=1000 * r["p10"], us_p90=1000 * r["p90"],
                achieved_gbs=r["gbs"] / world, pct_of_8TBps=100 * r["gbs"] / world / NOMINAL_HBM_GBS,
                algorithmic_mb=r["bytes"]["total"] / 1e6, note=note)
            del op_h
        # the same layer and cache under the paper's own index setting (512 lists, eight 4-bit
        # subspaces = 4 bytes of codes per token, 4 sinks, 128-token window, budget in whole
        # pages): every number the paper prints uses it
        cfg_p = dataclasses.replace(cfg, name=cfg.name.replace("c3", "c3p", 1), n_list=512, pq_m=8,
                                    pq_ncode=16, n_sink=4, n_local=128, exact_set_multiple=16)
        inp_p = dataclasses.replace(inp, cfg=cfg_p)
        idx_p = build_index(inp_p)
        op_p = DecodeOp(inp_p, idx_p, device=dev)
        r = measure(op_p, cfg_p, cfg_p.budget_ppm, args.steps, args.warmup, list(cfg_p.seq_lens))
        variants[cfg_p.name] = dict(
            us_per_step=1000 * r["ms"], us_p10=1000 * r["p10"], us_p90=1000 * r["p90"],
            achieved_gbs=r["gbs"] / world, pct_of_8TBps=100 * r["gbs"] / world / NOMINAL_HBM_GBS,
            algorithmic_mb=r["bytes"]["total"] / 1e6,
            index="n_list 512, 8 subspaces x 4 bits, 4 sinks, 128-token window, page-rounded budget")
        del op_p, idx_p

    # the other configurations of the benchmark plan, each generated, indexed and timed on its
    # own: the 32K layer, the ragged G = 8 batch, and three points of the context sweep with the
    # dense comparator beside them (time of the library's dense kernel, and of one read of K and
    # V at the measured copy rate)
    if not args.no_variants and cfg.name.startswith("c3") and world == 1:
        for name in ("c2", "c4", "c5_n16_b1", "c5_n128_b1", "c5_n512_b1"):
            torch.cuda.empty_cache()
            cfg_x = dataclasses.replace(parse_workload(name), kmeans_iters=min(2, args.kmeans_iters))
            inp_x = generate(cfg_x, device=dev)
            idx_x = build_index(inp_x)
            op_x = DecodeOp(inp_x, idx_x, device=dev)
            steps_x = max(10, args.steps // 4)
            r = measure(op_x, cfg_x, cfg_x.budget_ppm, steps_x, 3, list(cfg_x.seq_lens))
            ent = dict(us_per_step=1000 * r["ms"], us_p10=1000 * r["p10"], us_p90=1000 * r["p90"],
                       achieved_gbs=r["gbs"], pct_of_measured_peak=100 * r["gbs"] / peak,
                       algorithmic_mb=r["bytes"]["total"] / 1e6, batch=cfg_x.batch,
                       context=cfg_x.max_seq_len, n_list=cfg_x.n_list, steps=steps_x)
            if name.startswith("c5"):
                dws_x = torch.empty(pqhsa.dense_workspace_bytes(op_x.params), dtype=torch.uint8, device=dev)
                dout_x = torch.empty_like(op_x.q)
                for _ in range(3):
                    pqhsa.dense_decode(op_x.params, op_x.q, op_x.kv, op_x.seq_lens, dout_x, dws_x)
                pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                         for _ in range(steps_x)]
                barrier()
                for a, b in pairs:
                    flush.zero_()
                    a.record()
                    pqhsa.dense_decode(op_x.params, op_x.q, op_x.kv, op_x.seq_lens, dout_x, dws_x)
                    b.record()
                barrier()
                d_ms = sum(a.elapsed_time(b) for a, b in pairs) / len(pairs)
                db = dense_attention_bytes(cfg_x, list(cfg_x.seq_lens))
                ent.update(dense_us=1000 * d_ms, ideal_dense_us=db / peak / 1e3,
                           dense_over_pqhsa=d_ms / r["ms"],
                           ideal_dense_over_pqhsa=(db / peak / 1e6) / r["ms"])
                del dws_x, dout_x
            variants[name] = ent
            del op_x, idx_x, inp_x
        torch.cuda.empty_cache()

    # dense comparator: the library's own split-K dense decode kernel over the same paged cache
    dws = torch.empty(pqhsa.dense_workspace_bytes(op.params), dtype=torch.uint8, device=dev)
    dout = torch.empty_like(op.q)
    for _ in range(3):
        pqhsa.dense_decode(op.params, op.q, op.kv, op.seq_lens, dout, dws)
    dsteps = max(5, args.steps // 4)
    dev_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                 for _ in range(dsteps)]
    barrier()
    for a, b in dev_pairs:
        flush.zero_()
        a.record()
        pqhsa.dense_decode(op.params, op.q, op.kv, op.seq_lens, dout, dws)
        b.record()
    barrier()
    dense_ms = reduce_max(sum(a.elapsed_time(b) for a, b in dev_pairs) / dsteps)
    dbytes = dense_attention_bytes(cfg, seq_lens)
    dense = dict(us_per_step=1000 * dense_ms, achieved_gbs=dbytes / (dense_ms * 1e-3) / 1e9,
                 bytes=dbytes, speedup_over_dense=dense_ms / head["ms"],
                 ideal_us_at_measured_peak=dbytes / peak / 1e3,
                 speedup_over_ideal_dense=(dbytes / peak / 1e6) / head["ms"],
                 kernel="dense_decode_kernel (own split-K dense decode attention, same cache)")

    # the same step replayed from a CUDA graph (no per-launch host work)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        op.decode()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    with torch.cuda.graph(graph, stream=side):
        op.decode()
    g_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
    barrier()
    for a, b in g_pairs:
        flush.zero_()
        a.record()
        graph.replay()
        b.record()
    barrier()
    graph_ms = reduce_max(sum(a.elapsed_time(b) for a, b in g_pairs) / len(g_pairs))

    # index maintenance (not part of the step): re-encode the last 256 tokens of every sequence
    # into the existing lists on a copy of the index arrays; amortised over the 256 steps
    # between two updates
    upd = None
    n_upd = min(256, min(seq_lens))
    if n_upd > 0:
        codes2, ids2, norms2 = op.codes.clone(), op.list_ids.clone(), op.key_norms.clone()
        vm2, cnt2 = op.list_vmeans.clone(), idx.list_counts.to(dev).clone()
        rw = pqhsa.make_index_rw(op.centroids, op.codebooks, codes2, ids2, norms2, vm2, cnt2)
        first = torch.tensor([n - n_upd for n in seq_lens], dtype=torch.int32, device=dev)
        cnt_new = torch.full((cfg.batch,), n_upd, dtype=torch.int32, device=dev)
        u_pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(5)]
        pqhsa.index_update(op.params, rw, op.kv, first, cnt_new, n_upd)
        barrier()
        for a, b in u_pairs:
            flush.zero_()
            a.record()
            pqhsa.index_update(op.params, rw, op.kv, first, cnt_new, n_upd)
            b.record()
        barrier()
        upd_ms = reduce_max(sum(a.elapsed_time(b) for a, b in u_pairs) / len(u_pairs))
        upd = dict(us_per_call=1000 * upd_ms, new_tokens_per_sequence=n_upd,
                   us_per_step_amortised=1000 * upd_ms / 256,
                   note="pqhsa_index_update: encode into the existing lists and refresh the list "
                        "means; the paper runs it every 256 steps")
        del codes2, ids2, norms2, vm2, cnt2

    # index build (not part of the step): the library's batched build of one layer's worth of
    # heads (sequence 0: all KV heads at once), paper's schedule of one coarse and two codebook
    # iterations, against the per-head builder on the same input
    build = None
    if rank == 0 and world == 1 and not args.no_variants:
        from paper_2609_33746_b200.index_builder import build_index_batched
        cfg_b = dataclasses.replace(cfg, batch=1, seq_lens=cfg.seq_lens[:1], kmeans_iters=1, pq_iters=2)
        inp_b = dataclasses.replace(inp, cfg=cfg_b, q=inp.q[:1], block_table=inp.block_table[:1],
                                    seq_lens=inp.seq_lens[:1])
        build_index_batched(inp_b)                    # warm-up (workspace allocation, first launch)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        build_index_batched(inp_b)
        torch.cuda.synchronize()
        t_batched = time.perf_counter() - t0
        t0 = time.perf_counter()
        build_index(inp_b)
        torch.cuda.synchronize()
        t_head = time.perf_counter() - t0
        build = dict(ms_per_layer_batched=1000 * t_batched, ms_per_layer_per_head=1000 * t_head,
                     heads=cfg_b.n_kv_heads, tokens=cfg_b.seq_lens[0], n_list=cfg_b.n_list,
                     pq_m=cfg_b.pq_m, iterations="1 coarse + 2 codebook",
                     seconds_for_32_layers=32 * t_batched,
                     context_only="paper: 0.84 s batched vs 6.53 s per head for 32 layers at 128K "
                                  "on one H20 (512 lists, eight 4-bit subspaces)")

    clocks = sampler.stop()              # sampled over every timed loop above
    try:      # an auxiliary figure: never let it cost the JSON line
        if clocks.get("sm_mhz"):
            sp = roofline["data_pipe"]
            n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
            cycles = stage_ms[1] * 1e-3 * clocks["sm_mhz"] * 1e6
            sp["table_reads_frac_of_one_wavefront_per_sm_clock"] = (
                sp["table_wavefronts_per_tile"] * sp["tiles_per_launch"] / n_sm / cycles)
    except Exception:
        pass
    cpu_baseline = None
    if rank == 0 and world == 1:
        # whole sequences (all query heads), one after the other, until about 10 s of oracle time
        from helpers import oracle_arrays_for_sequence
        dt, nbytes, n_seq = 0.0, 0.0, 0
        for b in range(cfg.batch):
            d, nb = oracle_sample(inp, oracle_arrays_for_sequence(inp, idx, b), cfg, cfg.budget_ppm,
                                  cfg.n_q_heads)
            dt += d
            nbytes += nb
            n_seq += 1
            if dt >= args.oracle_seconds:
                break
        cpu_baseline = dict(value=nbytes / dt / 1e9, unit="GB/s", cores=cpu_threads(),
                            kind="oracle", seconds=dt, host_cpus=os.cpu_count(),
                            sample=f"float64 numpy oracle, sequences 0..{n_seq - 1} of {cfg.batch}, "
                                   f"all {cfg.n_q_heads} query heads ({n_seq / cfg.batch:.3f} of one "
                                   f"step), {dt:.1f} s")

    if rank == 0:
        n_tok = sum(seq_lens)
        line = dict(
            metric=METRIC, value=head["gbs"], unit="GB/s", n_gpus=world, steps=args.steps,
            warmup=args.warmup, ms_per_step=head["ms"], higher_is_better=True, scaling="weak",
            vs_baseline=None, dtype="f32", data="synthetic",
            config=dict(workload=cfg.name, batch=cfg.batch, context=cfg.max_seq_len,
                        n_q_heads=cfg.n_q_heads, n_kv_heads=cfg.n_kv_heads, head_dim=cfg.head_dim,
                        kv_dtype=cfg.dtype, page_size=cfg.page_size, n_list=cfg.n_list,
                        pq_m=cfg.pq_m, budget_ppm=cfg.budget_ppm, kmeans_iters=cfg.kmeans_iters,
                        l2="flushed between steps by a 512 MiB device write (not timed); "
                           "per-step CUDA events on the launch stream",
                        input_generation_s=round(t_gen, 1)),
            us_per_step=1000 * head["ms"], us_p10=1000 * head["p10"], us_p50=1000 * head["p50"],
            us_p90=1000 * head["p90"],
            pct_of_8TBps=100 * head["gbs"] / world / NOMINAL_HBM_GBS,
            pct_of_measured_peak=100 * head["gbs"] / world / peak,
            decode_tokens_per_s=world * cfg.batch / (head["ms"] * 1e-3),
            key_tokens_scanned_per_s=world * cfg.n_kv_heads * n_tok / (head["ms"] * 1e-3),
            algorithmic_bytes_per_step=head["bytes"], dense_attention_bytes=dense_attention_bytes(cfg, seq_lens),
            clocks=clocks, e2e=e2e, gpu_launches=launches, roofline=roofline,
            cpu_baseline=cpu_baseline, variants=variants, dense_comparator=dense,
            graph_replay_us_per_step=1000 * graph_ms, index_update=upd, index_build=build,
            context_only="paper: 1.58x over FlashAttention-3 on one H20 at 128K, 1% (other "
                         "hardware, other index setting)")
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
