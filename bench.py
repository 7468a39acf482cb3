"""Benchmark of the append-prefill hot path of one sparse layer: indexer -> top-k -> page demand -> sparse attention.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C] [--impl ours|reference]

A step is one pass of the whole path over one synthetic session (the exact pass; the predicted pass that feeds the
miss set is prepared once, untimed).  Metric: new tokens/s per sparse layer.  Prints ONE JSON line (rank 0).
With N > 1 (torchrun) every rank runs its own session (independent problems, no data-path collective): weak scaling.
--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "append_prefill_new_tokens_per_sec_per_sparse_layer"
UNIT = "tokens/s"


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"], "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.skip = 0
        self.proc = None

    def start(self):
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "25", "-i", str(self.index)],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def wait_until_running(self, timeout_s: float = 10.0):
        """Blocks until nvidia-smi has delivered its first sample, then forgets the samples taken so far: its start-up
        (driver initialisation on every GPU of the box) otherwise falls into the warm-up or timed steps and shows up as a
        multi-millisecond gap inside whichever kernel is running, and an idle sample is not a sample under load."""
        if self.proc is None:
            return
        t0 = time.time()
        while not self.rows and time.time() - t0 < timeout_s and self.proc.poll() is None:
            time.sleep(0.02)
        self.skip = len(self.rows)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows[self.skip:]:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None, "reasons": sorted(reasons),
                "samples": len(sm)}


def probe_fp8_peak(seconds: float = 1.0):
    """Dense FP8 tensor rate of this GPU, measured outside the timed region (TFLOP/s): the library's own tcgen05 loop
    (operands in shared memory, M = 128, N = 256, the indexer's instruction shape) and, as a library cross-check, a
    torch._scaled_mm E4M3 GEMM of 8192^3.  `burst` = best of several short launches; `sustained` = back to back for about
    `seconds` (the rate the power limit allows, which is what a kernel inside a long step sees)."""
    import torch
    from paper_2609_36938_b200 import binding as B

    ev = lambda: torch.cuda.Event(enable_timing=True)
    out = {}
    n_sm = torch.cuda.get_device_properties(torch.cuda.current_device()).multi_processor_count

    def timed(fn, flop, reps):
        e0, e1 = ev(), ev()
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return flop * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12, e0.elapsed_time(e1) * 1e-3

    fills = 4096                                             # 5.1 TFLOP per launch, under 2 ms
    flop = 2.0 * 128 * 256 * 128 * fills * n_sm
    own = lambda: B.janus_fp8_mma_probe(n_sm, fills)
    own(); torch.cuda.synchronize()
    out["own_loop_burst"] = max(timed(own, flop, 1)[0] for _ in range(10))
    rate, dt = timed(own, flop, 50)
    reps = max(50, int(50 * seconds / dt))
    out["own_loop_sustained"] = timed(own, flop, reps)[0]
    B.check_dev_status()
    try:
        n = 8192
        a = torch.randn((n, n), device="cuda").to(torch.float8_e4m3fn)
        b = torch.randn((n, n), device="cuda").to(torch.float8_e4m3fn).t()     # column-major second operand
        one = torch.ones((), device="cuda")
        mm = lambda: torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        mm(); torch.cuda.synchronize()
        gflop = 2.0 * n * n * n
        out["scaled_mm_burst"] = max(timed(mm, gflop, 1)[0] for _ in range(10))
        rate, dt = timed(mm, gflop, 50)
        out["scaled_mm_sustained"] = timed(mm, gflop, max(50, int(50 * seconds / dt)))[0]
        del a, b
    except Exception as e:      # the probe is a cross-check only
        out["scaled_mm_error"] = f"{type(e).__name__}: {e}"[:200]
    return {k: (round(v, 1) if isinstance(v, float) else v) for k, v in out.items()}


def captured_traffic(kernel_key: str, rows: int):
    """DRAM bytes of one launch of `kernel_key`, from the ncu capture summarised under profiles/ (a small case of the same
    kernel), scaled by query rows to this launch.  None if no capture is recorded."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if not os.path.exists(p):
        return None
    e = json.load(open(p)).get("dram_bytes_per_launch", {}).get(kernel_key)
    return None if e is None else e["bytes"] * rows / e["rows"]


def workload_numbers(shp):
    """Algorithmic work of one step (exact pass): flops and bytes each call must do at least, from the shapes alone."""
    L, M, S = shp.L, shp.M, shp.S
    pairs = M * L + M * (M + 1) // 2
    sel = sum(min(shp.k, L + t + 1) for t in range(M))
    esz = 2 if shp.idx_dtype == "bf16" else 1
    row_bytes = shp.d_qk * 2 if shp.attn == "latent" else (shp.d_qk + shp.d_v) * 2 * shp.n_kv_heads
    return {
        "pairs": pairs,
        "indexer_flops": 2.0 * shp.H_I * shp.D_I * pairs,
        "indexer_bytes": esz * (M * shp.H_I * shp.D_I + S * shp.D_I) + 4 * M * shp.H_I + 4.0 * pairs,
        "topk_bytes": 4.0 * pairs + 4.0 * M * shp.k,
        "page_demand_bytes": 4.0 * M * shp.k,
        "attn_flops": 2.0 * shp.H_q * (shp.d_qk + shp.d_v) * sel,
        "attn_bytes": float(row_bytes) * sel + 2.0 * M * shp.H_q * (shp.d_qk + shp.d_v),
        "selected_rows": sel,
    }


def run_reference(args, shp, sess):
    """The CPU oracle, as it stands, on a bounded sample of query rows of the same workload."""
    from oracle import janus_oracle as O
    from paper_2609_36938_b200 import workloads as W

    n_rows = args.ref_rows
    rows = W.sample_rows(shp.M, n_rows)

    def step():
        sc = O.indexer_scores(sess["q_idx"], sess["k_idx"], sess["w"], dtype=shp.idx_dtype, q_scale=sess["q_scale"], k_scale=sess["k_scale"],
                              recency=sess["recency"], q_pos0=shp.L, causal=True, rows=rows)
        idx = O.topk(sc, shp.k, q_pos0=shp.L, causal=True, rows=rows)
        O.page_demand(idx, shp.L, shp.page_size, sess["page_table"])
        O.sparse_attention(sess["Q"], sess["k_pool"], sess["v_pool"], sess["page_table"], idx, page_size=shp.page_size,
                           softmax_scale=shp.softmax_scale, d_qk=shp.d_qk, d_v=shp.d_v, rows=rows)

    # The oracle's matrix products run in the BLAS numpy links; a launcher that exports OMP_NUM_THREADS=1 (torchrun does)
    # would pin it to one thread, so the thread count is set here to the cores this process may use, and reported.
    cores = len(os.sched_getaffinity(0))
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        limiter = threadpool_limits(limits=cores)
    except Exception:
        limiter, threadpool_info = None, None
    for _ in range(args.warmup_ref):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps_ref):
        step()
    dt = (time.perf_counter() - t0) / args.steps_ref
    if threadpool_info is not None:
        used = [int(p.get("num_threads", 0)) for p in threadpool_info() if p.get("user_api") in ("blas", "openmp")]
        if used:
            cores = max(used)
    if limiter is not None:
        limiter.restore_original_limits()
    value = len(rows) / dt
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{len(rows)} of {shp.M} query rows (first, last, evenly spread), all {shp.S} keys, k={shp.k}; "
                      f"rows are independent, rows/s reported as tokens/s", "ms_per_step": dt * 1e3}


def run_decode(args):
    """Side workload (not the headline metric): one decode step over `--decode-batch` sessions of `--L` cached tokens each
    (default 131072), FP8 64 x 128 indexer, latent attention, k = 2048.  Inputs are made on the device (parity of this
    path is covered by tests/test_gpu_decode.py); prints one JSON line with per-call times and the indexer's bandwidth."""
    import torch
    from paper_2609_36938_b200 import binding as B, build as _build

    torch.cuda.set_device(0)
    _build.build()
    B.load()
    nb, L, k, page, H, D = args.decode_batch, (args.L or 131072), 2048, 64, 64, 128
    g = torch.Generator(device="cuda").manual_seed(args.seed)
    n_keys = (L + 1 + 3) // 4 * 4
    key_off = torch.arange(nb + 1, dtype=torch.int64, device="cuda") * n_keys
    row_len = torch.full((nb,), L + 1, dtype=torch.int64, device="cuda")
    fp4 = args.decode_fp4_keys
    k_idx = torch.randint(0, 256, (nb * n_keys, D // 2 if fp4 else D), dtype=torch.uint8, device="cuda", generator=g)
    if not fp4:
        k_idx = torch.where((k_idx & 0x7f) >= 0x7f, k_idx & 0xf7, k_idx)      # no NaN codes
    q_idx = torch.randint(0, 120, (nb, H, D), dtype=torch.uint8, device="cuda", generator=g)
    w = torch.rand((nb, H), device="cuda", generator=g) / 8
    q_scale = torch.ones((nb, H), device="cuda") / 64
    k_scale = torch.ones((nb * n_keys,), device="cuda") / 64
    pages_per = (L + 1 + page - 1) // page
    n_phys = nb * pages_per
    tables = torch.randperm(n_phys, device="cuda", generator=g).int()
    tab_off = torch.arange(nb + 1, dtype=torch.int64, device="cuda") * pages_per
    limits = torch.full((nb,), L, dtype=torch.int64, device="cuda")
    pool = (torch.randn((n_phys, page, 1, 576), device="cuda", generator=g) / 24).bfloat16()
    q = (torch.randn((nb, 128, 576), device="cuda", generator=g) / 24).bfloat16()
    scores = torch.empty((nb * n_keys,), dtype=torch.float32, device="cuda")
    ev = lambda: torch.cuda.Event(enable_timing=True)

    def step(marks=None):
        if marks: marks[0].record()
        B.janus_indexer_scores_batch(q_idx, k_idx, w, key_off, n_keys, q_scale=q_scale, k_scale=k_scale, scores=scores, keys_fp4=fp4)
        if marks: marks[1].record()
        idx, _, _ = B.janus_topk_batch(scores, key_off, k, row_lengths=row_len, want_count=False, want_kth=False)
        if marks: marks[2].record()
        pd = B.janus_page_demand_batch(idx, demand_limits=limits, page_size=page, page_tables=tables, table_offsets=tab_off, n_phys_pages=n_phys)
        if marks: marks[3].record()
        out, _ = B.janus_sparse_attn_decode(q, pool, pool, idx, page_tables=tables, table_offsets=tab_off, page_size=page,
                                            softmax_scale=1 / 24, d_v=512, want_lse=False)
        if marks: marks[4].record()
        return out

    for _ in range(max(args.warmup, 3)):
        step()
    B.check_dev_status()
    marks = [[ev() for _ in range(5)] for _ in range(args.steps)]
    torch.cuda.synchronize()
    for m in marks:
        step(m)
    torch.cuda.synchronize()
    B.check_dev_status()
    per = np.array([[m[j].elapsed_time(m[j + 1]) for j in range(4)] for m in marks]).mean(axis=0)
    total_ms = float(np.mean([m[0].elapsed_time(m[4]) for m in marks]))
    peaks = load_peaks()
    key_bytes = nb * (L + 1) * ((D // 2 if fp4 else D) + 4 + 4)   # key row + its scale read, score written
    line = {"metric": "decode_tokens_per_sec_per_sparse_layer", "value": nb / (total_ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
            "steps": args.steps, "ms_per_step": total_ms, "data": "synthetic (device-generated)", "dtype": "fp8_e4m3+bf16",
            "config": {"workload": f"decode step: {nb} sessions x {L} cached tokens, k={k}, {'FP8 queries / FP4 keys' if fp4 else 'FP8'} 64x128 indexer, latent attention, page {page}"},
            "kernels": {"indexer_scores_batch": {"ms": float(per[0]), "gbs": key_bytes / (per[0] * 1e-3) / 1e9,
                                                 "frac_hbm_peak": key_bytes / (per[0] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
                        "topk_batch": {"ms": float(per[1]), "gbs": nb * (L + 1) * 4 / (per[1] * 1e-3) / 1e9},
                        "page_demand_batch": {"ms": float(per[2])},
                        "sparse_attn_decode": {"ms": float(per[3]), "logical_gbs": nb * k * 1152 / (per[3] * 1e-3) / 1e9}}}
    print(json.dumps(line))


def run_sharded_prediction(args, rank, world, local_rank):
    """--shard keys: the synchronisation-free parallel prediction of Sec. 4.2 (Eq. 3) across ranks.  Every rank holds the
    lookahead queries and its own disjoint, page-aligned shard C_n of the history keys; a step is indexer -> top-(k/N) ->
    page demand on that shard (no exchange: the rank could start prefetching its pages here) followed by the one
    exchange of the partition, the union of the ranks' page bitmaps that the exact pass is compared against.  The whole
    job's work is fixed (one session's prediction pass), so scaling is strong.  The session is the first one of the
    ragged batch (config 4), the configuration whose predicted set is defined."""
    import torch
    import torch.distributed as dist

    from paper_2609_36938_b200 import binding as B, build as _build, dist_utils as D, prediction as P, report as R, workloads as W

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    B.load()
    shp = W.batch_shapes(args.seed)[0] if (args.L is None and args.M is None) else W.config_shape(4, L=args.L, M=args.M)
    sess = W.make_session(shp, args.seed, with_attention=False, page_table=W.make_page_table(
        W.config_shape(2, L=shp.L, M=shp.M), args.seed), n_phys_pages=shp.n_logical_pages)
    n_phys = sess["n_phys_pages"]
    kind = shp.idx_dtype
    bounds = P.shard_bounds(shp.L, world, shp.page_size)
    a, b = bounds[rank] if rank < len(bounds) else (0, 0)
    k_shard = max(1, shp.k // world)
    q_pred = B.to_device(sess["q_pred"], kind)
    w = B.to_device(sess["w"], "f32")
    k_mine = B.to_device(sess["k_idx"][a:b], kind)
    table = B.to_device(sess["page_table"], "i32")
    table_mine = table[a // shp.page_size:]
    ld = ((b - a) + 31) // 32 * 32
    scores = torch.empty((shp.M, max(ld, 32)), dtype=torch.float32, device="cuda")
    idx = torch.empty((shp.M, k_shard), dtype=torch.int32, device="cuda")
    bufs = B.page_demand_buffers(n_phys, want_miss=False)
    union_fn = lambda dst, src: B.janus_page_union(dst, src, n_phys)

    def step():
        sc = B.janus_indexer_scores(q_pred, k_mine, w, q_pos0=shp.L, causal=False, scores=scores)
        B.janus_topk(sc, b - a, k_shard, q_pos0=shp.L, causal=False, want_count=False, want_kth=False, idx=idx)
        pd = B.janus_page_demand(idx, demand_limit=b - a, page_size=shp.page_size, page_table=table_mine, n_phys_pages=n_phys, want_miss=False, out=bufs)
        return D.or_reduce_bitmap(pd["bitmap"], union_fn)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_until_running()
    for _ in range(max(args.warmup, 3)):
        union = step()
    B.check_dev_status()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        union = step()
    e1.record()
    barrier()
    B.check_dev_status()
    # strong scaling: every rank reports the whole session's M tokens once (rank 0 only), the time is the maximum over ranks
    value, elapsed_ms, _ = D.aggregate_throughput(float(shp.M * args.steps) if rank == 0 else 0.0, e0.elapsed_time(e1), device="cuda")
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0:
        # untimed: the exact pass of the same session on this rank, and what the united prediction covers of it
        k_all = B.to_device(sess["k_idx"], kind)
        sc = B.janus_indexer_scores(B.to_device(sess["q_idx"], kind), k_all, w, q_pos0=shp.L, causal=True)
        eidx, _, _ = B.janus_topk(sc, shp.S, shp.k, q_pos0=shp.L, causal=True, want_count=False, want_kth=False)
        pd = B.janus_page_demand(eidx, demand_limit=shp.L, page_size=shp.page_size, page_table=table, n_phys_pages=n_phys, predicted_bitmap=union)
        rep = R.demand_report(pd, union)
        B.check_dev_status()
        line = {"metric": "sharded_prediction_new_tokens_per_sec_per_sparse_layer", "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": max(args.warmup, 3), "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
                "dtype": kind, "data": "synthetic", "clocks": clocks,
                "config": {"workload": f"key-sharded prediction pass (Eq. 3): L={shp.L} M={shp.M} k={shp.k} -> top-{k_shard} per shard, {world} page-aligned "
                                       f"history shards, indexer {shp.H_I}x{shp.D_I} {kind}, page {shp.page_size}, shuffled page table",
                           "exchange": "one all-gather of the page bitmaps + local union (janus_page_union) per step"},
                "gpu_launches": 5 * args.steps, "page_report_vs_exact": rep}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_query_sharded(args, rank, world, local_rank):
    """--shard queries: the query-parallel partition (Sec. 4.2): query rows are independent, so rank n runs the whole exact
    pass (indexer -> top-k -> page demand -> attention) on its contiguous slice of the M new tokens against replicated keys and
    KV pool; the only exchange is the union of the ranks' page bitmaps (one all-gather + janus_page_union), from which every
    rank has the session's page demand.  Total work is fixed: strong scaling."""
    import torch
    import torch.distributed as dist

    from paper_2609_36938_b200 import binding as B, build as _build, dist_utils as D, workloads as W

    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    B.load()
    shp = W.config_shape(args.workload if args.workload != 4 else 3, L=args.L, M=args.M)
    sess = W.make_session(shp, args.seed)                      # the same session on every rank
    kind = shp.idx_dtype
    r0, r1 = rank * shp.M // world, (rank + 1) * shp.M // world
    m = r1 - r0
    n_keys = shp.L + r1                                        # keys the last row of the slice may see
    dev = lambda name, kd, sl=slice(None): None if sess[name] is None else B.to_device(sess[name][sl], kd)
    q_idx, w, Q = dev("q_idx", kind, slice(r0, r1)), dev("w", "f32", slice(r0, r1)), dev("Q", "bf16", slice(r0, r1))
    k_idx, k_scale, col_bias = dev("k_idx", kind, slice(0, n_keys)), dev("k_scale", "f32", slice(0, n_keys)), dev("col_bias", "f32", slice(0, n_keys))
    q_scale, row_bias = dev("q_scale", "f32"), dev("row_bias", "f32", slice(r0, r1))
    table, pool = dev("page_table", "i32"), dev("k_pool", "bf16")
    n_phys = sess["n_phys_pages"]
    ld = (n_keys + 31) // 32 * 32
    scores = torch.empty((max(m, 1), ld), dtype=torch.float32, device="cuda")
    idx = torch.empty((max(m, 1), shp.k), dtype=torch.int32, device="cuda")
    out = torch.empty((max(m, 1), shp.H_q, shp.d_v), dtype=torch.bfloat16, device="cuda")
    bufs = B.page_demand_buffers(n_phys, want_miss=False)
    union_fn = lambda dst, src: B.janus_page_union(dst, src, n_phys)

    def step():
        if m > 0:
            sc = B.janus_indexer_scores(q_idx, k_idx, w, q_scale=q_scale, k_scale=k_scale, row_bias=row_bias, col_bias=col_bias, q_pos0=shp.L + r0,
                                        causal=True, scores=scores)
            B.janus_topk(sc, n_keys, shp.k, q_pos0=shp.L + r0, causal=True, want_count=False, want_kth=False, idx=idx)
            pd = B.janus_page_demand(idx, demand_limit=shp.L, page_size=shp.page_size, page_table=table, n_phys_pages=n_phys, want_miss=False, out=bufs)
            B.janus_sparse_attn_prefill(Q, pool, pool, idx, page_table=table, page_size=shp.page_size, softmax_scale=shp.softmax_scale, d_v=shp.d_v,
                                        want_lse=False, out=out)
            bm = pd["bitmap"]
        else:
            bm = torch.zeros_like(bufs["bitmap"])
        return D.or_reduce_bitmap(bm, union_fn)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        sampler.wait_until_running()
    for _ in range(max(args.warmup, 3)):
        union = step()
    B.check_dev_status()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        union = step()
    e1.record()
    barrier()
    B.check_dev_status()
    value, elapsed_ms, _ = D.aggregate_throughput(float(shp.M * args.steps) if rank == 0 else 0.0, e0.elapsed_time(e1), device="cuda")
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0:
        from paper_2609_36938_b200 import report as R
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
                "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
                "dtype": "fp8_e4m3+bf16" if kind == "fp8" else "bf16", "data": "synthetic", "clocks": clocks,
                "config": {"workload": f"query-sharded exact pass: L={shp.L} M={shp.M} k={shp.k} split into {world} contiguous row slices, keys and KV pool "
                                       f"replicated, indexer {shp.H_I}x{shp.D_I} {kind}, latent attention, page {shp.page_size}",
                           "exchange": "one all-gather of the page bitmaps + local union (janus_page_union) per step"},
                "gpu_launches": 5 * args.steps, "union_pages": R.popcount(union)}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, help="benchmark configuration 1..5 (4 = the ragged batch of 8 sessions, one after another)")
    ap.add_argument("--sessions", type=int, default=None, help="with --workload 4: only the first N sessions of the batch")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--L", type=int, default=None)
    ap.add_argument("--M", type=int, default=None)
    ap.add_argument("--ref-rows", type=int, default=16)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-fused", action="store_true", help="skip the side measurement of janus_indexer_topk")
    ap.add_argument("--no-peak-probe", action="store_true", help="skip the FP8 tensor-rate probe (the roofline then divides by an assumed peak)")
    ap.add_argument("--no-report", action="store_true", help="skip the recall / precision / run-length report of configs 1, 4, 5")
    ap.add_argument("--shard", default="none", choices=["none", "keys", "queries"],
                    help="with --gpus N: keys = time the key-sharded prediction pass (Eq. 3): rank n scores its own history shard; "
                         "queries = rank n runs the exact pass on its slice of the new tokens; either way one union of page bitmaps")
    ap.add_argument("--decode-batch", type=int, default=0, help="side workload: time one decode step over this many sessions instead")
    ap.add_argument("--decode-fp4-keys", action="store_true", help="with --decode-batch: indexer keys stored as FP4 E2M1")
    args = ap.parse_args()
    if args.decode_batch > 0:
        run_decode(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    args.steps_ref = max(1, min(args.steps, 3))
    args.warmup_ref = 1 if args.warmup > 0 else 0

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.shard == "keys" and args.impl == "ours":
        run_sharded_prediction(args, rank, world, local_rank)
        return
    if args.shard == "queries" and args.impl == "ours":
        run_query_sharded(args, rank, world, local_rank)
        return

    from paper_2609_36938_b200 import workloads as W

    if args.workload == 4 and args.L is None and args.M is None:
        shapes = W.batch_shapes(args.seed)
        if args.sessions:
            shapes = shapes[:args.sessions]
    else:
        shapes = [W.config_shape(args.workload, L=args.L, M=args.M)]
    n_sessions = len(shapes)
    shp = shapes[0]
    if n_sessions == 1:
        sizes = f"L={shp.L} M={shp.M}"
    else:
        sizes = f"{n_sessions} sessions one after another, L={[x.L for x in shapes]} M={[x.M for x in shapes]}"
    workload_name = (f"config {args.workload}: {sizes} k={shp.k}, indexer {shp.H_I}x{shp.D_I} {shp.idx_dtype}, "
                     f"{shp.attn} attention {shp.H_q} heads {shp.d_qk}/{shp.d_v} bf16, page {shp.page_size}, {shp.table} page table")
    config = {"workload": workload_name, "sessions_per_gpu": n_sessions, "cache": "inputs larger than L2 (scores, Q and gathered KV are GBs per step)"}

    def make_sessions(seed):
        if n_sessions > 1 or shp.table == "fragmented":
            return W.make_batch(seed, shapes)
        return [W.make_session(shp, seed)]

    if args.impl == "reference":
        if rank != 0:
            return
        sess = make_sessions(args.seed)[0]
        cb = run_reference(args, shp, sess)
        if n_sessions > 1:
            cb["sample"] = "first session of the batch: " + cb["sample"]
        line = {"metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps_ref, "warmup": args.warmup_ref,
                "ms_per_step": cb["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
                "data": "synthetic", "config": config, "impl": "reference",
                "cpu_baseline": {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")},
                "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(line))
        return

    import torch
    import torch.distributed as dist

    from paper_2609_36938_b200 import binding as B, build as _build, dist_utils as D, report as R

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl")
    if rank == 0:
        _build.build()
    if world > 1:
        dist.barrier()
    B.load()

    sessions = make_sessions(args.seed + rank)
    kind = shp.idx_dtype
    tokens_per_step = sum(x.M for x in shapes)
    n_phys = sessions[0]["n_phys_pages"]

    # pinned host copies of every operand; tensors shared by sessions (the KV pool of a batch) are held, uploaded and counted once
    pinned_by_id = {}

    def pin(arr, kd):
        if arr is None:
            return None
        if id(arr) not in pinned_by_id:
            pinned_by_id[id(arr)] = B.to_device(arr, kd, device="cpu").pin_memory()
        return pinned_by_id[id(arr)]

    pinned = []
    for sess in sessions:
        pinned.append({
            "q_idx": pin(sess["q_idx"], kind), "k_idx": pin(sess["k_idx"], kind), "w": pin(sess["w"], "f32"), "q_scale": pin(sess["q_scale"], "f32"),
            "k_scale": pin(sess["k_scale"], "f32"), "row_bias": pin(sess["row_bias"], "f32"), "col_bias": pin(sess["col_bias"], "f32"),
            "page_table": pin(sess["page_table"], "i32"), "Q": pin(sess["Q"], "bf16"), "k_pool": pin(sess["k_pool"], "bf16"),
            "v_pool": pin(sess["v_pool"], "bf16"),
        })
    h2d_bytes = sum(t.numel() * t.element_size() for t in pinned_by_id.values())

    def device_set():
        """One device copy of every distinct pinned tensor, and the per-session views onto them."""
        dev_by_id = {i: torch.empty_like(t, device="cuda") for i, t in pinned_by_id.items()}
        by_pin = {id(t): dev_by_id[i] for i, t in pinned_by_id.items()}
        views = [{n: (None if t is None else by_pin[id(t)]) for n, t in pn.items()} for pn in pinned]
        return dev_by_id, views

    def upload_all(dev_by_id):
        for i, t in pinned_by_id.items():
            dev_by_id[i].copy_(t, non_blocking=True)

    dev0, d_list = device_set()
    upload_all(dev0)
    ld_max = max((x.S + 31) // 32 * 32 for x in shapes)
    scores_buf = torch.empty((max(x.M for x in shapes) * ld_max,), dtype=torch.float32, device="cuda")
    out_bufs = [torch.empty((x.M, x.H_q, x.d_v), dtype=torch.bfloat16, device="cuda") for x in shapes]
    idx_bufs = [torch.empty((x.M, x.k), dtype=torch.int32, device="cuda") for x in shapes]

    def scores_view(x):
        ld = (x.S + 31) // 32 * 32
        return scores_buf[:x.M * ld].view(x.M, ld)

    # predicted pass (Eq. 2): same indexer on the lookahead queries over the history keys only; prepared once per session
    pred_bitmaps, pred_idx = [], []
    for x, sess, d in zip(shapes, sessions, d_list):
        if "q_pred" not in sess:
            pred_bitmaps.append(None); pred_idx.append(None)
            continue
        qp = B.to_device(sess["q_pred"], kind)
        psc = B.janus_indexer_scores(qp, d["k_idx"][:x.L], d["w"], q_scale=d["q_scale"],
                                     k_scale=None if d["k_scale"] is None else d["k_scale"][:x.L], q_pos0=x.L, causal=False)
        pidx, _, _ = B.janus_topk(psc, x.L, x.k, q_pos0=x.L, causal=False, want_count=False, want_kth=False)
        pred_bitmaps.append(B.janus_page_demand(pidx, demand_limit=x.L, page_size=x.page_size, page_table=d["page_table"],
                                                n_phys_pages=n_phys, want_miss=False)["bitmap"])
        pred_idx.append(pidx)
        del psc, qp
    torch.cuda.empty_cache()

    ev = lambda: torch.cuda.Event(enable_timing=True)
    stream = torch.cuda.current_stream()
    pd_bufs = [B.page_demand_buffers(n_phys) for _ in shapes]      # allocated once: the timed path neither allocates nor fills

    def session_step(b, d, marks=None, out_to=None):
        """The four calls of the exact pass of session b on the device operands d."""
        x = shapes[b]
        if marks is not None:
            marks[0].record(stream)
        sc = B.janus_indexer_scores(d["q_idx"], d["k_idx"], d["w"], q_scale=d["q_scale"], k_scale=d["k_scale"], row_bias=d["row_bias"],
                                    col_bias=d["col_bias"], q_pos0=x.L, causal=True, scores=scores_view(x))
        if marks is not None:
            marks[1].record(stream)
        idx, _, _ = B.janus_topk(sc, x.S, x.k, q_pos0=x.L, causal=True, want_count=False, want_kth=False, idx=idx_bufs[b])
        if marks is not None:
            marks[2].record(stream)
        pd = B.janus_page_demand(idx, demand_limit=x.L, page_size=x.page_size, page_table=d["page_table"], n_phys_pages=n_phys,
                                 predicted_bitmap=pred_bitmaps[b], out=pd_bufs[b])
        if marks is not None:
            marks[3].record(stream)
        out, _ = B.janus_sparse_attn_prefill(d["Q"], d["k_pool"], d["v_pool"], idx, page_table=d["page_table"], page_size=x.page_size,
                                             softmax_scale=x.softmax_scale, d_v=x.d_v, want_lse=False, out=out_bufs[b] if out_to is None else out_to)
        if marks is not None:
            marks[4].record(stream)
        return idx, pd, out

    def step(marks=None):
        res = None
        for b in range(n_sessions):
            res = session_step(b, d_list[b], None if marks is None else marks[b])
        return res

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local_rank)      # runs through warm-up, the timed region and the end-to-end region (all under load)
    if rank == 0:
        sampler.start()
        sampler.wait_until_running()
    if world > 1:
        dist.barrier()
    for _ in range(args.warmup):
        step()
    B.check_dev_status()

    # ---- timed region: device-resident inputs
    marks = [[[ev() for _ in range(5)] for _ in range(n_sessions)] for _ in range(args.steps)]
    barrier()
    t_start, t_end = ev(), ev()
    t_start.record(stream)
    for i in range(args.steps):
        idx, pd, out = step(marks[i])
    t_end.record(stream)
    barrier()
    B.check_dev_status()
    elapsed_ms = t_start.elapsed_time(t_end)
    # [steps, 4] ms: per call, summed over the sessions of a step
    per_call = np.array([[sum(m[b][j].elapsed_time(m[b][j + 1]) for b in range(n_sessions)) for j in range(4)] for m in marks])
    per_session_ms = [float(np.mean([m[b][0].elapsed_time(m[b][4]) for m in marks])) for b in range(n_sessions)]
    value, elapsed_ms, _ = D.aggregate_throughput(float(tokens_per_step * args.steps), elapsed_ms, device="cuda")   # max over ranks
    ms_per_step = elapsed_ms / args.steps

    # ---- end to end: every step uploads all inputs from pinned host memory and reads the results back
    e2e = None
    if not args.no_e2e:
        host_out = [torch.empty(o.shape, dtype=o.dtype).pin_memory() for o in out_bufs]
        host_idx = [torch.empty(ib.shape, dtype=torch.int32).pin_memory() for ib in idx_bufs]
        host_pages = torch.empty((n_phys,), dtype=torch.int32).pin_memory()
        host_counts = torch.empty((4,), dtype=torch.int32).pin_memory()
        d2h_bytes = sum(t.numel() * t.element_size() for t in host_out + host_idx) + n_sessions * (host_pages.numel() + 4) * 4

        # Three streams, two sets of device buffers: the upload of step i+1 and the read-back of step i-1 run while step i
        # computes, as a serving loop would do it.  Every step still copies all of its inputs from pinned host memory and
        # all of its results back; the timed region covers all of it.
        s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
        dev_sets = [device_set() for _ in range(2)]
        dev_out = [[torch.empty_like(o) for o in out_bufs] for _ in range(2)]
        in_done = [ev() for _ in range(2)]
        cmp_done = [ev() for _ in range(2)]
        out_done = [ev() for _ in range(2)]

        def e2e_steps(n):
            for i in range(n):
                s2 = i & 1
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(cmp_done[s2])          # step i-2 has finished reading this input set
                    upload_all(dev_sets[s2][0])
                    in_done[s2].record(s_in)
                with torch.cuda.stream(s_cmp):
                    s_cmp.wait_event(in_done[s2])
                    if i >= 2:
                        s_cmp.wait_event(out_done[s2])         # step i-2's output buffers have been read back
                    results = [session_step(b, dev_sets[s2][1][b], out_to=dev_out[s2][b]) for b in range(n_sessions)]
                    cmp_done[s2].record(s_cmp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(cmp_done[s2])
                    for b, (ridx, rpd, rout) in enumerate(results):
                        host_out[b].copy_(rout, non_blocking=True)
                        host_idx[b].copy_(ridx, non_blocking=True)
                        host_pages.copy_(rpd["pages"][:n_phys], non_blocking=True)
                        host_counts.copy_(rpd["counts"], non_blocking=True)
                    out_done[s2].record(s_out)
            for st in (s_in, s_cmp, s_out):
                stream.wait_stream(st)

        e2e_steps(2)
        barrier()
        e0, e1 = ev(), ev()
        n_e2e = max(4, min(args.steps, 8))
        e0.record(stream)
        for st in (s_in, s_cmp, s_out):
            st.wait_stream(stream)
        e2e_steps(n_e2e)
        e1.record(stream)
        barrier()
        e2e_value, e2e_total_ms, _ = D.aggregate_throughput(float(tokens_per_step * n_e2e), e0.elapsed_time(e1), device="cuda")
        e2e_ms = e2e_total_ms / n_e2e
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d_bytes), "d2h_bytes_per_step": int(d2h_bytes),
               "ms_per_step": e2e_ms, "inputs": "all operands (queries, keys, weights, Q, KV pool, page table) uploaded every step; upload, compute and read-back of "
                         "consecutive steps overlap on three streams (two buffer sets)"}
        del dev_sets, dev_out
        torch.cuda.empty_cache()

    # a short run can end between two samples: keep the same load on until one sample has been taken under it
    if rank == 0 and sampler.proc is not None:
        t_wait = time.time()
        while len(sampler.rows) - sampler.skip < 2 and time.time() - t_wait < 2.0:
            step()
            torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None

    # ---- report (untimed, from the device outputs of the last step): recall / precision of the predicted page set against the
    # exact one, miss-set size, runs, the same at token granularity, and the run-length histogram (shuffled and identity table)
    report = None
    if rank == 0 and not args.no_report and (args.workload in (1, 4, 5)):
        report = {"sessions": []}
        for b, x in enumerate(shapes):
            r = {"L": x.L, "M": x.M, "pages": R.demand_report(pd_bufs[b], pred_bitmaps[b]),
                 "tokens": R.token_granularity_report(idx_bufs[b], pred_idx[b], x.L)}
            if args.workload == 5 or n_sessions == 1:
                r["run_length_histogram"] = {str(k_): v for k_, v in sorted(R.run_length_histogram(pd_bufs[b]).items())}
                ident = torch.arange(x.n_logical_pages, dtype=torch.int32, device="cuda")
                pd_id = B.janus_page_demand(idx_bufs[b], demand_limit=x.L, page_size=x.page_size, page_table=ident, n_phys_pages=x.n_logical_pages, want_miss=False)
                r["identity_table"] = {"n_runs": int(pd_id["counts"][1].item()), "n_pages": int(pd_id["counts"][0].item()),
                                       "run_length_histogram": {str(k_): v for k_, v in sorted(R.run_length_histogram(pd_id).items())}}
            report["sessions"].append(r)
        if any(p_ is not None for p_ in pred_bitmaps):
            for level in ("pages", "tokens"):
                report[f"mean_{level}_recall"] = float(np.mean([r[level]["recall"] for r in report["sessions"]]))
                report[f"mean_{level}_precision"] = float(np.mean([r[level]["precision"] for r in report["sessions"]]))
                report[f"mean_{level}_miss"] = float(np.mean([r[level]["n_miss"] for r in report["sessions"]]))
        B.check_dev_status()

    # ---- side measurement (not part of `value`): indexer + top-k as one call that never stores the score matrix
    fused = None
    if not args.no_fused and n_sessions == 1:
        lib = B.load()
        d = d_list[0]
        ws_bytes = int(lib.janus_indexer_topk_workspace_size(shp.M, shp.H_I, shp.D_I, shp.S, shp.L, 1, 1 if shp.idx_dtype == "fp8" else 0, shp.k))
        del scores_buf
        torch.cuda.empty_cache()
        ws = torch.empty((ws_bytes,), dtype=torch.uint8, device="cuda")
        fidx = torch.empty((shp.M, shp.k), dtype=torch.int32, device="cuda")

        def fused_call():
            B.janus_indexer_topk(d["q_idx"], d["k_idx"], d["w"], shp.k, q_scale=d["q_scale"], k_scale=d["k_scale"], row_bias=d["row_bias"],
                                 col_bias=d["col_bias"], q_pos0=shp.L, causal=True, workspace=ws, idx=fidx, want_count=False, want_kth=False)

        for _ in range(3):
            fused_call()
        barrier()
        f0, f1 = ev(), ev()
        f0.record(stream)
        for _ in range(5):
            fused_call()
        f1.record(stream)
        barrier()
        B.check_dev_status()
        fused = {"ms": f0.elapsed_time(f1) / 5, "two_call_ms": float(per_call[:, 0].mean() + per_call[:, 1].mean()), "workspace_bytes": ws_bytes,
                 "score_matrix_bytes": int(shp.M) * int((shp.S + 31) // 32 * 32) * 4,
                 "note": "one call that never stores the score matrix: a memory-saving path (workspace vs score matrix), not the faster one at this size"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = load_peaks()
    wns = [workload_numbers(x) for x in shapes]
    wn = {k_: sum(w_[k_] for w_ in wns) for k_ in wns[0]}
    mean_ms = per_call.mean(axis=0)
    names = ["indexer_scores", "topk", "page_demand", "sparse_attn_prefill"]
    fp8 = shp.idx_dtype == "fp8"
    # FP8 tensor peak: measured in this run (sustained: the indexer runs inside a long step); the larger of the library's own
    # tcgen05 loop and the torch._scaled_mm GEMM, so that the fraction is never flattered.  Twice the measured bf16 figure
    # (the nominal ratio) is kept beside it.
    fp8_probe = None
    assumed_fp8 = peaks["bf16_tflops_sustained"] * 2.0
    if fp8 and not args.no_peak_probe:
        fp8_probe = probe_fp8_peak()
        fp8_probe["assumed_2x_bf16_sustained"] = assumed_fp8
    if fp8:
        if fp8_probe is not None:
            tensor_peak_idx = max(fp8_probe.get("own_loop_sustained", 0.0), fp8_probe.get("scaled_mm_sustained", 0.0))
            peak_source_idx = ("measured in this run: sustained dense FP8 E4M3 rate, max of the library's own tcgen05 loop "
                               f"({fp8_probe.get('own_loop_sustained')} TFLOP/s) and torch._scaled_mm 8192^3 ({fp8_probe.get('scaled_mm_sustained')} TFLOP/s)")
        else:
            tensor_peak_idx = assumed_fp8
            peak_source_idx = f"ASSUMED: {peaks['source']} bf16 sustained x2 (nominal fp8:bf16 ratio); no FP8 probe in this run"
    else:
        tensor_peak_idx = peaks["bf16_tflops_sustained"]
        peak_source_idx = f"{peaks['source']} bf16 sustained"
    rows_total = sum(x.M for x in shapes)
    attn_dram = captured_traffic("sparse_attn_latent", rows_total) if shp.attn == "latent" else None
    kernels = {
        "indexer_scores": {"ms": mean_ms[0], "tflops": wn["indexer_flops"] / (mean_ms[0] * 1e-3) / 1e12,
                           "frac_tensor_peak": wn["indexer_flops"] / (mean_ms[0] * 1e-3) / 1e12 / tensor_peak_idx},
        "topk": {"ms": mean_ms[1], "gbs": wn["topk_bytes"] / (mean_ms[1] * 1e-3) / 1e9,
                 "frac_hbm_peak": wn["topk_bytes"] / (mean_ms[1] * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "page_demand": {"ms": mean_ms[2], "gbs": wn["page_demand_bytes"] / (mean_ms[2] * 1e-3) / 1e9},
        "sparse_attn_prefill": {"ms": mean_ms[3], "tflops": wn["attn_flops"] / (mean_ms[3] * 1e-3) / 1e12,
                                "logical_gbs": wn["attn_bytes"] / (mean_ms[3] * 1e-3) / 1e9,
                                "frac_hbm_peak_logical": wn["attn_bytes"] / (mean_ms[3] * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                "frac_tensor_peak": wn["attn_flops"] / (mean_ms[3] * 1e-3) / 1e12 / peaks["bf16_tflops_sustained"]},
    }
    if attn_dram is not None:    # what actually came from DRAM (ncu capture, scaled by rows): most gathered rows are L2 hits
        kernels["sparse_attn_prefill"]["dram_gbs_captured"] = attn_dram / (mean_ms[3] * 1e-3) / 1e9
        kernels["sparse_attn_prefill"]["frac_hbm_peak_dram"] = attn_dram / (mean_ms[3] * 1e-3) / 1e9 / peaks["hbm_gbs"]
    kernels["topk_plus_gather"] = {"ms": mean_ms[1] + mean_ms[3], "logical_gbs": (wn["topk_bytes"] + wn["attn_bytes"]) / ((mean_ms[1] + mean_ms[3]) * 1e-3) / 1e9,
                                   "frac_hbm_peak_logical": (wn["topk_bytes"] + wn["attn_bytes"]) / ((mean_ms[1] + mean_ms[3]) * 1e-3) / 1e9 / peaks["hbm_gbs"]}
    dom = int(np.argmax(mean_ms))
    if names[dom] == "indexer_scores":
        roofline = {"kernel": "indexer_tc_kernel", "bound": "tensor", "achieved": kernels["indexer_scores"]["tflops"], "peak": tensor_peak_idx,
                    "unit": "TFLOP/s", "frac": kernels["indexer_scores"]["frac_tensor_peak"],
                    "traffic": captured_traffic("indexer_tc" if fp8 else "indexer_tc_bf16", rows_total),
                    "traffic_note": "ncu dram bytes of a smaller capture of the same kernel scaled by rows (profiles/traffic.json)",
                    "peak_source": peak_source_idx}
        if fp8_probe is not None:
            roofline["frac_of_assumed_2x_bf16_sustained"] = kernels["indexer_scores"]["tflops"] / assumed_fp8
            roofline["frac_of_measured_fp8_burst"] = kernels["indexer_scores"]["tflops"] / max(fp8_probe.get("own_loop_burst", 0.0), fp8_probe.get("scaled_mm_burst", 1e-9))
    elif names[dom] == "sparse_attn_prefill":
        roofline = {"kernel": "sparse_attn", "bound": "tensor", "achieved": kernels["sparse_attn_prefill"]["tflops"],
                    "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s", "frac": kernels["sparse_attn_prefill"]["frac_tensor_peak"],
                    "traffic": attn_dram, "peak_source": f"{peaks['source']} bf16 sustained"}
    else:
        key = names[dom]
        roofline = {"kernel": key, "bound": "hbm", "achieved": kernels[key]["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": kernels[key]["gbs"] / peaks["hbm_gbs"], "traffic": captured_traffic("topk_rows" if key == "topk" else "page_mark", rows_total),
                    "peak_source": f"{peaks['source']} copy bandwidth"}

    cpu_baseline = None
    if not args.no_cpu_baseline:
        cb = run_reference(args, shp, sessions[0])
        if n_sessions > 1:
            cb["sample"] = "first session of the batch: " + cb["sample"]
        cpu_baseline = {k: cb[k] for k in ("value", "unit", "cores", "kind", "sample")}

    counts = pd["counts"].cpu().numpy()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3+bf16" if fp8 else "bf16", "data": "synthetic",
        "config": config, "clocks": clocks, "e2e": e2e,
        # kernels of this library per session pass: indexer, top-k, page mark, page lists, attention (plus one cudaMemsetAsync of the bitmap)
        "gpu_launches": 5 * args.steps * n_sessions, "roofline": roofline, "cpu_baseline": cpu_baseline, "fp8_peak_probe": fp8_probe,
        "kernels": {k: {kk: (round(float(vv), 4)) for kk, vv in v.items()} for k, v in kernels.items()},
        "indexer_topk_one_call": fused,
        "page_demand": {"n_pages": int(counts[0]), "n_runs": int(counts[1]), "n_miss": int(counts[2]), "n_miss_runs": int(counts[3])},
    }
    if n_sessions > 1:
        line["ms_per_session"] = [round(v, 4) for v in per_session_ms]
    if report is not None:
        line["report"] = report
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
