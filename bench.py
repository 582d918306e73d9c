#!/usr/bin/env python
"""Benchmark of the SparseD attention hot path on B200.

One "step" is one pass of the whole hot path over one synthetic batch of the 64k workload:
schedule helper -> dense attention that also records per-tile row statistics -> pattern
selection from those statistics (pooling to A', isolated top-k, CSR) -> block-sparse attention
on the selected pattern. The headline value is the block-sparse
attention throughput in TFLOP/s counted on kept-block FLOPs (4 * bs^2 * D * nnz), with its
fraction of the measured bf16 peak and the wall-time speedup over the library's own dense
kernel reported beside it.

    python bench.py --gpus 1 --steps 5 --warmup 3            # this library
    python bench.py --impl reference --steps 2 --warmup 1     # the CPU oracle on host cores

With --gpus N > 1 (under torchrun) every rank runs an independent replica of the workload
(the path has no exchange step); value = work of all ranks / max-over-ranks time.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2509_24014_b200 import replicas  # noqa: E402
from paper_2509_24014_b200 import synthetic as syn  # noqa: E402

METRIC = "block-sparse attn TFLOP/s, % bf16 peak, speedup vs own dense kernel at 64k"

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from ncu captures of the
# kernels, keyed by (kernel, workload): (bytes, where the figure comes from, source file of the kernel,
# sha256 prefix of that file when the capture was taken). A figure whose kernel source has changed
# since is reported as null with the reason, instead of going stale silently.
_C2_ATTN = "ncu --set full capture of one launch on the 8k workload (summary under profiles/)"
_C2_POOL = "ncu --set full capture of one launch on the 8k workload (summary under profiles/)"
_ATTN_SRC = ("paper_2509_24014_b200/csrc/attention.cu", "paper_2509_24014_b200/csrc/softmax_pipeline.cuh",
             "paper_2509_24014_b200/csrc/sm100_primitives.cuh")
_ATTN_SHA = "258d6b93c29d"
_PAIR_SRC = ("paper_2509_24014_b200/csrc/attention_dense_pair.cu", "paper_2509_24014_b200/csrc/sm100_pair_primitives.cuh",
             "paper_2509_24014_b200/csrc/softmax_pipeline.cuh", "paper_2509_24014_b200/csrc/sm100_primitives.cuh",
             "paper_2509_24014_b200/build.py")   # (its compile flags are set per file there)
_PAIR_SHA = "ac9c2ae83227"
_POOL_SRC = ("paper_2509_24014_b200/csrc/pool_select.cu", "paper_2509_24014_b200/csrc/topk_device.cuh")
_POOL_SHA = "2a48dbebbbc2"
NCU_DRAM_TRAFFIC = {
    ("attn_dense_pair_kernel", "c2"): (201576192 + 102648320, _C2_ATTN, _PAIR_SRC, _PAIR_SHA),
    ("attn_kernel<sparse>", "c2"): (156466176 + 43784192, _C2_ATTN, _ATTN_SRC, _ATTN_SHA),
    ("pool_select_kernel", "c2"): (68194816 + 587776, _C2_POOL, _POOL_SRC, _POOL_SHA),
    # 64k workload: the 8k capture scaled by the algorithmic bytes of a launch (traffic was the algorithmic
    # traffic at 8k: every K/V re-read hits L2), instead of a multi-counter capture of a 7 GB workload.
    # dense + statistics: Q,K,V,O + LSE + statistics = 6450 MB at 64k against 336 MB at 8k
    ("attn_dense_pair_kernel", "c4"): (int((201576192 + 102648320) * 6450.0 / 336.0), _C2_ATTN + ", scaled x19.2 by algorithmic bytes",
                                       _PAIR_SRC, _PAIR_SHA),
    # sparse: Q + O + touched K,V: 8x the rows and 8x the K/V of the 8k workload
    ("attn_kernel<sparse>", "c4"): ((156466176 + 43784192) * 8, _C2_ATTN + ", scaled x8 by algorithmic bytes",
                                    _ATTN_SRC, _ATTN_SHA),
    # pooling: the statistics stream, 64x the 8k one (rows x8, key blocks x8)
    ("pool_select_kernel", "c4"): ((68194816 + 587776) * 64, _C2_POOL + ", scaled x64 by algorithmic bytes",
                                   _POOL_SRC, _POOL_SHA),
}


def _source_digest(rel_paths):
    """sha256 prefix over the named source files (a kernel may be spread over several)."""
    import hashlib
    h = hashlib.sha256()
    try:
        for rel in rel_paths:
            with open(os.path.join(ROOT, rel), "rb") as f:
                h.update(f.read())
    except OSError:
        return None
    return h.hexdigest()[:12]


def ncu_traffic(kernel, workload):
    """(bytes or None, provenance string) for roofline.traffic."""
    rec = NCU_DRAM_TRAFFIC.get((kernel, workload))
    if rec is None:
        return None, "no ncu capture for this kernel and workload"
    nbytes, where, src, digest = rec
    if _source_digest(src) != digest:
        return None, f"stale: {' / '.join(src)} changed since the capture ({where})"
    return nbytes, where


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.lines = []      # (arrival time, text)
        self.proc = None
        self.t_begin = 0.0

    def mark_begin(self):
        """Samples that arrive before this moment (warm-up) are not counted."""
        self.t_begin = time.monotonic()

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.monotonic(), line.strip()))

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for t_line, ln in self.lines:
            if t_line < self.t_begin:
                continue
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1])); power.append(float(parts[2]))
            except ValueError:
                continue
            for n, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def sparse_flops(cfg, nnz):
    return 4.0 * cfg.block_size * cfg.block_size * cfg.head_dim * nnz


def dense_flops(cfg):
    return 4.0 * cfg.seq_len * cfg.seq_len * cfg.head_dim * cfg.heads_q * cfg.batch


# ------------------------------------------------------------------------------ CPU oracle leg
def oracle_sparse_sample(cfg, q, k, v, rp, ci, n_row_blocks, seed=0):
    """Times the fp64 oracle's masked attention on a seeded sample of (head, query block) rows.
    Returns (kept-block TFLOP/s, seconds, rows, threads)."""
    from oracle import sparsed_oracle as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    rng = np.random.default_rng(seed)
    nb = cfg.num_blocks
    group = cfg.heads_q // cfg.heads_kv
    heads = rng.integers(0, cfg.heads_q, n_row_blocks)
    blocks = rng.integers(0, nb, n_row_blocks)
    cache = {}
    flops = 0.0
    t_total = 0.0
    for h, ib in zip(heads, blocks):
        hk = int(h) // group
        if ("k", hk) not in cache:
            cache.clear()
            cache[("k", hk)] = (k[0, hk].to(torch.float64).numpy(), v[0, hk].to(torch.float64).numpy())
        kh, vh = cache[("k", hk)]
        qh = q[0, int(h)].to(torch.float64).numpy()
        r = int(h) * nb + int(ib)
        kept = ci[rp[r]:rp[r + 1]]
        t0 = time.perf_counter()
        orc.head_sparse_rows(qh, kh, vh, int(ib), kept, cfg.block_size)
        t_total += time.perf_counter() - t0
        flops += 4.0 * cfg.block_size * cfg.block_size * cfg.head_dim * len(kept)
    return flops / t_total / 1e12, t_total, n_row_blocks, threads


def oracle_stage_samples(cfg, q, k, v, n_row_blocks, seed=1):
    """Times the oracle's other stages (full attention; pooled scoring + selection) on a seeded
    sample of (head, query block) rows and extrapolates to the whole workload (the work per row
    block is uniform). Returns a dict for the cpu_baseline record."""
    from oracle import sparsed_oracle as orc
    rng = np.random.default_rng(seed)
    nb, bs = cfg.num_blocks, cfg.block_size
    group = cfg.heads_q // cfg.heads_kv
    pb = cfg.prefill_len // bs
    h = int(rng.integers(0, cfg.heads_q))
    qh = q[0, h].to(torch.float64).numpy()
    kh = k[0, h // group].to(torch.float64).numpy()
    vh = v[0, h // group].to(torch.float64).numpy()
    blocks = [int(x) for x in rng.integers(0, nb, n_row_blocks)]
    t0 = time.perf_counter()
    for ib in blocks:
        orc.head_full_rows(qh, kh, vh, slice(ib * bs, (ib + 1) * bs))
    t_full = time.perf_counter() - t0
    t0 = time.perf_counter()
    for ib in blocks:
        orc.select_row(orc.head_pooled_row(qh, kh, ib, bs), pb, cfg.keep_ratio)
    t_sel = time.perf_counter() - t0
    total_rows = cfg.batch * cfg.heads_q * nb
    scale = total_rows / n_row_blocks
    return {"rows_sampled": n_row_blocks, "rows_total": total_rows,
            "attn_full": {"cpu_seconds_sample": t_full, "cpu_seconds_extrapolated": t_full * scale,
                          "tflops": 4.0 * bs * cfg.seq_len * cfg.head_dim * n_row_blocks / t_full / 1e12},
            "score_and_select": {"cpu_seconds_sample": t_sel, "cpu_seconds_extrapolated": t_sel * scale}}


def run_reference(args, cfg):
    """The oracle as it stands, timed on the host cores, on bounded samples of the workload."""
    from oracle import sparsed_oracle as orc
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    small = cfg.with_(heads_q=2, heads_kv=2 if cfg.heads_kv == cfg.heads_q else 1)
    q, k, v = syn.make_qkv(small, "cpu")
    nb = cfg.num_blocks
    pb = cfg.prefill_len // cfg.block_size
    k_pre, k_gen = orc.kept_per_region(pb, cfg.keep_ratio), orc.kept_per_region(nb - pb, cfg.keep_ratio)
    kh, vh = k[0, 0].to(torch.float64).numpy(), v[0, 0].to(torch.float64).numpy()
    qh = q[0, 0].to(torch.float64).numpy()
    rows_per_step = args.ref_rows
    rng = np.random.default_rng(0)

    def one_step():
        flops = 0.0
        for _ in range(rows_per_step):
            ib = int(rng.integers(0, nb))
            # select this row block's pattern with the oracle itself, then attend
            kept = orc.select_row(orc.head_pooled_row(qh, kh, ib, cfg.block_size), pb, cfg.keep_ratio)
            t0 = time.perf_counter()
            orc.head_sparse_rows(qh, kh, vh, ib, kept, cfg.block_size)
            one_step.sparse_s += time.perf_counter() - t0
            flops += 4.0 * cfg.block_size ** 2 * cfg.head_dim * len(kept)
        return flops

    one_step.sparse_s = 0.0
    for _ in range(args.warmup):
        one_step()
    one_step.sparse_s = 0.0
    t0 = time.perf_counter()
    flops = 0.0
    for _ in range(args.steps):
        flops += one_step()
    wall = time.perf_counter() - t0
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = os.cpu_count() or 1
    value = flops / one_step.sparse_s / 1e12
    sample = (f"{rows_per_step} seeded (head, query block) rows of {cfg.heads_q * nb} per step; each row: oracle "
              f"scoring+selection (untimed) then oracle masked attention (timed), k={k_pre}+{k_gen} of {nb} blocks")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": wall / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": bench_config(cfg, k_pre, k_gen, args.gpus), "timing": "host perf_counter",
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


def bench_config(cfg, k_pre, k_gen, world=1, shard_heads=False):
    """The `config` object of the JSON line; the same for this library's arm and the reference arm."""
    nb = cfg.num_blocks
    nnz = cfg.batch * cfg.heads_q * nb * (k_pre + k_gen)
    qkvo_gb = 2.0 * cfg.batch * cfg.seq_len * cfg.head_dim * (2 * cfg.heads_q + 2 * cfg.heads_kv) / 1e9
    return {"workload": workload_name(cfg), "step": "attn_full_stats -> select_from_stats -> attn_sparse",
            "kept_per_row": [k_pre, k_gen], "nnz": nnz, "density": nnz / (cfg.batch * cfg.heads_q * nb * nb),
            "l2": "inputs larger than L2 (Q,K,V,O = %.2f GB per pass)" % qkvo_gb,
            "parallelism": ("heads sharded over ranks, no collective" if shard_heads else
                            "replicas only" if world > 1 else "single GPU")}


def workload_name(cfg):
    return (f"{cfg.name}: B{cfg.batch} Hq{cfg.heads_q}/Hkv{cfg.heads_kv} L{cfg.seq_len} D{cfg.head_dim} bf16, "
            f"block {cfg.block_size}, keep {cfg.keep_ratio}, prefill {cfg.prefill_len}")


# ------------------------------------------------------------------------------ GPU arm
def _ev():
    return torch.cuda.Event(enable_timing=True)


def slow_path_events(ws):
    """Warp-level rescales of the output accumulator counted by the attention kernels in the workspace."""
    return int(ws[32:40].view(torch.int64).item())


def measure_config(cfg, dev, layer=0, qkv=None):
    """Buffers and the step closure of the hot path on one workload, resident in HBM: a step is
    attn_full_stats -> select_from_stats -> attn_sparse, optionally dropping four CUDA events.
    cfg describes the tensors this rank holds; qkv overrides the synthetic inputs (head shards)."""
    import paper_2509_24014_b200 as sd
    q, k, v = qkv if qkv is not None else syn.make_qkv(cfg, dev, layer)
    B, Hq, L, D = q.shape
    bs, nb = cfg.block_size, cfg.num_blocks
    o_full = torch.empty_like(q)
    o_sparse = torch.empty_like(q)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=dev)
    params = sd.make_params(bs, cfg.keep_ratio, cfg.prefill_len)
    k_pre, k_gen = sd.sparsed_kept_per_row(params, L)
    pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
    shape_qkvo = sd.make_shape(q, k, v, o_full)
    shape_qk = sd.make_shape(q, k)
    ws = sd.new_workspace(256, dev)
    tile_stats = sd.new_tile_stats(q, bs)

    def step(marks=None):
        def mark():
            if marks is not None:
                e = _ev(); e.record(); marks.append(e)
        mark()
        sd.sparsed_attn_full_stats(q, k, v, o_full, lse, tile_stats, ws, bs, shape=shape_qkvo)
        mark()
        sd.sparsed_select_from_stats(q, k, params, lse, tile_stats, pat, ws, shape=shape_qk)
        mark()
        sd.sparsed_attn_sparse(q, k, v, o_sparse, pat, ws, shape=shape_qkvo)
        mark()

    return {"q": q, "k": k, "v": v, "o_full": o_full, "o_sparse": o_sparse, "lse": lse, "params": params,
            "kept": (k_pre, k_gen), "pat": pat, "row_ptr": row_ptr, "col_idx": col_idx, "ws": ws,
            "tile_stats": tile_stats, "step": step, "shape_qkvo": shape_qkvo, "shape_qk": shape_qk}


def time_config(cfg, dev, reps, warmup, peaks, layer=0):
    """measure_config + timing, for the by-config summary. Frees the workload before returning."""
    import paper_2509_24014_b200 as sd
    m = measure_config(cfg, dev, layer)
    for _ in range(warmup):
        m["step"]()
    torch.cuda.synchronize()
    events = []
    for _ in range(reps):
        marks = []
        m["step"](marks)
        events.append(marks)
    a, b = _ev(), _ev()
    a.record()
    for _ in range(reps):
        sd.sparsed_attn_full(m["q"], m["k"], m["v"], m["o_full"], None, m["ws"], shape=m["shape_qkvo"])
    b.record()
    torch.cuda.synchronize()
    code, where = sd.sparsed_last_device_status(m["ws"])
    if code != 0:
        raise RuntimeError(f"device status {code} at {where}")
    full_stats_ms = statistics.median(e[0].elapsed_time(e[1]) for e in events)
    select_ms = statistics.median(e[1].elapsed_time(e[2]) for e in events)
    sparse_ms = statistics.median(e[2].elapsed_time(e[3]) for e in events)
    dense_ms = a.elapsed_time(b) / reps
    nnz = int(m["pat"].nnz)
    k_pre, k_gen = m["kept"]
    nb = cfg.num_blocks
    peak = peaks["bf16_tflops"]
    sparse_tf = sparse_flops(cfg, nnz) / sparse_ms / 1e9
    dense_tf = dense_flops(cfg) / dense_ms / 1e9
    B, Hq, L, D = m["q"].shape
    # How often the softmax had to rescale its accumulator (logits outgrew the running maximum), per
    # warp-level softmax group (32 query rows x 64 keys), separately for the dense and the sparse kernel.
    sd.sparsed_workspace_init(m["ws"])
    sd.sparsed_attn_full(m["q"], m["k"], m["v"], m["o_full"], None, m["ws"], shape=m["shape_qkvo"])
    torch.cuda.synchronize()
    ev_dense = slow_path_events(m["ws"])
    sd.sparsed_attn_sparse(m["q"], m["k"], m["v"], m["o_sparse"], m["pat"], m["ws"], shape=m["shape_qkvo"])
    torch.cuda.synchronize()
    ev_sparse = slow_path_events(m["ws"]) - ev_dense
    groups_dense = B * Hq * ((L + 31) // 32) * ((L + 63) // 64)
    groups_sparse = nnz * max(1, cfg.block_size // 32) * max(1, cfg.block_size // 64)
    out = {"workload": workload_name(cfg), "plant_norm": cfg.plant_norm, "kept_per_row": [k_pre, k_gen], "nnz": nnz,
           "dense_ms": dense_ms, "dense_tflops": dense_tf, "dense_frac_of_burst": dense_tf / peak,
           "dense_with_stats_ms": full_stats_ms, "select_from_stats_ms": select_ms,
           "sparse_ms": sparse_ms, "sparse_tflops": sparse_tf, "sparse_frac_of_burst": sparse_tf / peak,
           "speedup_vs_dense": dense_ms / sparse_ms, "ideal_speedup": nb / (k_pre + k_gen),
           "softmax_rescale_fraction_dense": ev_dense / groups_dense,
           "softmax_rescale_fraction_sparse": ev_sparse / groups_sparse, "reps": reps}
    if cfg.block_size < 128 and nb % (128 // cfg.block_size) == 0:
        # packed walk: how much of each shared query tile's work is on blocks its own query block kept
        g = 128 // cfg.block_size
        kk = k_pre + k_gen
        ids = m["col_idx"][: B * Hq * nb * kk].view(B * Hq * (nb // g), g * kk).long()
        seen = torch.zeros(ids.shape[0], nb, dtype=torch.bool, device=dev)
        seen.scatter_(1, ids, True)
        union = seen.sum(dim=1).double()
        out["useful_fraction_of_tile_work"] = float((g * kk) / (g * union).mean().item() / 1.0) if union.numel() else None
        out["mean_union_blocks_per_tile"] = float(union.mean().item())
    return out


def run_ours(args, cfg):
    import paper_2509_24014_b200 as sd

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU fallback)")
    from paper_2509_24014_b200 import build as _build
    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        _build.build_library()   # compiles only if the library is missing or older than its sources
    else:
        for _ in range(600):     # other ranks wait for rank 0's build instead of racing it
            if not _build.is_stale():
                break
            time.sleep(0.5)
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    sd.load_library()
    peaks = load_peaks()

    shard_heads = args.shard == "heads" and world > 1
    if shard_heads:
        # one layer split over the ranks by heads (whole GQA groups): same seed everywhere, each rank
        # keeps its own heads; total work is fixed as N grows
        hq = replicas.shard_heads(cfg.heads_q, cfg.heads_kv, world, rank)
        hkv = replicas.shard_kv_heads(cfg.heads_kv, world, rank)
        qf, kf, vf = syn.make_qkv(cfg, dev)
        qkv = (qf[:, hq.start:hq.stop].contiguous(), kf[:, hkv.start:hkv.stop].contiguous(),
               vf[:, hkv.start:hkv.stop].contiguous())
        del qf, kf, vf
        torch.cuda.empty_cache()
        cfg_local = cfg.with_(heads_q=len(hq), heads_kv=len(hkv))
        m = measure_config(cfg_local, dev, qkv=qkv)
        del qkv
    else:
        cfg_local = cfg.with_(seed=replicas.replica_seed(cfg.seed, rank))
        m = measure_config(cfg_local, dev)
    q, k, v, o_full, o_sparse, lse = m["q"], m["k"], m["v"], m["o_full"], m["o_sparse"], m["lse"]
    B, Hq, L, D = q.shape
    nb = cfg.num_blocks
    params, pat, row_ptr, col_idx, ws = m["params"], m["pat"], m["row_ptr"], m["col_idx"], m["ws"]
    k_pre, k_gen = m["kept"]
    shape_qkvo, shape_qk, tile_stats = m["shape_qkvo"], m["shape_qk"], m["tile_stats"]
    total_steps, skip = max(cfg.total_steps, 2), (cfg.skip if cfg.total_steps > 1 else 0.5)
    s_switch = sd.sparsed_switch_step(total_steps, skip)
    assert sd.sparsed_schedule_mode(s_switch, total_steps, skip) == sd.MODE_FULL_AND_SELECT
    assert sd.sparsed_schedule_mode(s_switch + 1, total_steps, skip) == sd.MODE_SPARSE
    step = m["step"]

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()          # nvidia-smi needs a moment to start streaming: launch it before the warm-up
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.mark_begin()
    events = []
    t_begin, t_end = _ev(), _ev()
    t_begin.record()
    for _ in range(args.steps):
        marks = []
        step(marks)
        events.append(marks)
    t_end.record()
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    total_ms = t_begin.elapsed_time(t_end)
    code, where = sd.sparsed_last_device_status(ws)
    if code != 0:
        raise RuntimeError(f"device status {code} at {where}")

    full_ms = [e[0].elapsed_time(e[1]) for e in events]
    select_ms = [e[1].elapsed_time(e[2]) for e in events]
    sparse_ms = [e[2].elapsed_time(e[3]) for e in events]
    sparse_total = sum(sparse_ms)
    nnz = int(pat.nnz)

    # the plain dense kernel (no statistics), the same number of calls back to back: what the
    # sparse step's speedup is measured against
    a, b = _ev(), _ev()
    a.record()
    for _ in range(args.steps):
        sd.sparsed_attn_full(q, k, v, o_full, None, ws, shape=shape_qkvo)
    b.record()
    torch.cuda.synchronize()
    dense_plain_total = a.elapsed_time(b)

    # max over ranks of the timed quantities
    total_ms, sparse_total, full_total, select_total, dense_plain_total = replicas.max_over_ranks(
        [total_ms, sparse_total, sum(full_ms), sum(select_ms), dense_plain_total], dist, dev)

    n = args.steps
    cfg_work = cfg_local          # the work one rank did
    value = world * n * sparse_flops(cfg_work, nnz) / (sparse_total * 1e-3) / 1e12
    dense_tflops = world * n * dense_flops(cfg_work) / (dense_plain_total * 1e-3) / 1e12
    dense_stats_tflops = world * n * dense_flops(cfg_work) / (full_total * 1e-3) / 1e12
    per_gpu_sparse = value / world

    # ---- end to end through the public API with host buffers (rank-local, then max) -------
    e2e_steps = max(1, min(args.steps, 3))
    hq_, hk_, hv_ = (t.to("cpu").pin_memory() for t in (q, k, v))
    ho = torch.empty(o_sparse.shape, dtype=o_sparse.dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in (hq_, hk_, hv_))
    d2h = ho.numel() * ho.element_size()
    torch.cuda.synchronize()
    e0, e1 = _ev(), _ev()
    from paper_2509_24014_b200.host_api import HostSparseAttention
    host_plan = HostSparseAttention(hq_, hk_, row_ptr, col_idx, cfg.block_size, dev)
    def e2e_once():
        host_plan.run(hq_, hk_, hv_, ho)
    e2e_once()
    torch.cuda.synchronize()
    assert torch.equal(ho.to(dev), o_sparse), "host-buffer path disagrees with the resident path"
    assert all(st == (0, 0) for st in host_plan.device_status())
    if dist is not None:
        dist.barrier()
    e0.record()
    for _ in range(e2e_steps):
        e2e_once()
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = e0.elapsed_time(e1)
    e2e_ms = replicas.max_over_ranks([e2e_ms], dist, dev)[0]
    del host_plan
    e2e_value = world * e2e_steps * sparse_flops(cfg_work, nnz) / (e2e_ms * 1e-3) / 1e12

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak = peaks["bf16_tflops"]
    tag = "of measured" if peaks["source"] == "measured" else "of fallback"

    def tensor_roofline(name, flops_per_launch, ms_list, launches_per_step=1):
        ms = sum(ms_list) / (len(ms_list) * launches_per_step)
        ach = flops_per_launch / (ms * 1e-3) / 1e12
        traffic, source = ncu_traffic(name, cfg.name)
        return {"kernel": name, "bound": "tensor", "achieved": ach, "peak": peak, "unit": "TFLOP/s",
                "frac": ach / peak, "peak_source": f"bf16 burst, {tag}",
                "frac_of_sustained": ach / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
                "avg_launch_ms": ms, "traffic": traffic, "traffic_source": source}

    def topk_roofline():
        """The ranking/compaction kernel alone (sparsed_select_from_scores) on this workload's A',
        HBM-bound by design; L2 is flushed before each launch by writing a 512 MB buffer."""
        scores = torch.empty(B, Hq, nb, nb, dtype=torch.float32, device=dev)
        sd.sparsed_select_from_stats(q, k, params, lse, tile_stats, pat, ws, scores_out=scores, shape=shape_qk)
        flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
        pat2, rp2, ci2 = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
        times = []
        for _ in range(5):
            flush.fill_(1)
            a, b = _ev(), _ev()
            a.record()
            sd.sparsed_select_from_scores(scores, params, pat2, ws)
            b.record()
            torch.cuda.synchronize()
            times.append(a.elapsed_time(b))
        assert torch.equal(ci2, col_idx) and torch.equal(rp2, row_ptr)
        ms = min(times[1:])
        nbytes = B * Hq * (4 * nb * nb + 4 * nb * (k_pre + k_gen) + 4 * nb)
        ach = nbytes / (ms * 1e-3) / 1e9
        traffic, source = ncu_traffic("topk_csr_kernel", cfg.name)
        return {"kernel": "topk_csr_kernel (stand-alone, not in the step)", "bound": "hbm", "achieved": ach,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": ach / peaks["hbm_gbs"],
                "peak_source": f"HBM copy, {tag}", "avg_launch_ms": ms, "algorithmic_bytes": nbytes,
                "traffic": traffic, "traffic_source": source,
                "note": "event time of a single launch includes launch latency; L2 flushed before it"}

    # the dense pass of the step records row statistics: that entry point runs the CTA-pair kernel
    roof_dense = tensor_roofline("attn_dense_pair_kernel", dense_flops(cfg_work), full_ms)
    roof_sparse = tensor_roofline("attn_kernel<sparse>", sparse_flops(cfg_work, nnz), sparse_ms)
    launches_per_step = 3
    # selection from the recorded statistics is HBM-bound: it reads 4 * L * L / block_size bytes per head
    stats_bytes = tile_stats.numel() * 4 + lse.numel() * 4 + 4 * nnz + 4 * (B * Hq * nb + 1)
    sel_ms = sum(select_ms) / len(select_ms)
    sel_gbs = stats_bytes / (sel_ms * 1e-3) / 1e9
    traffic, source = ncu_traffic("pool_select_kernel", cfg.name)
    roof_select = {"kernel": "pool_select_kernel", "bound": "hbm", "achieved": sel_gbs, "peak": peaks["hbm_gbs"],
                   "unit": "GB/s", "frac": sel_gbs / peaks["hbm_gbs"], "peak_source": f"HBM copy, {tag}",
                   "avg_launch_ms": sel_ms, "algorithmic_bytes": stats_bytes,
                   "algorithmic_bytes_of_selection_alone": B * Hq * (4 * nb * nb + 4 * nb * (k_pre + k_gen) + 4 * nb),
                   "traffic": traffic, "traffic_source": source}
    roof_topk = topk_roofline() if not shard_heads else None
    dominant = max((roof_dense, roof_select, roof_sparse), key=lambda r: r["avg_launch_ms"])
    roof_all = [r for r in (roof_dense, roof_select, roof_sparse, roof_topk) if r is not None]

    # ---- CPU oracle beside it (bounded sample of the same workload) ----------------------
    cpu = None
    if not args.no_cpu_baseline:
        rp_h = row_ptr.cpu().numpy()
        ci_h = col_idx.cpu().numpy()
        n_rows = args.cpu_rows
        val, secs, rows, threads = oracle_sparse_sample(cfg_work, hq_, hk_, hv_, rp_h, ci_h, n_rows)
        cpu = {"value": val, "unit": "TFLOP/s", "cores": threads, "kind": "oracle",
               "sample": f"oracle masked attention (fp64 numpy) on {rows} seeded (head, query block) rows of "
                         f"{Hq * nb}, GPU-selected pattern, {secs:.1f} s; kept-block FLOPs / time",
               "seconds": secs, "host_cpus": os.cpu_count(),
               "cpu_seconds_extrapolated": secs * (B * Hq * nb) / rows,
               "gpu_ms": {"attn_full_stats": full_total / n, "select_from_stats": select_total / n,
                          "attn_sparse": sparse_total / n},
               "other_stages": oracle_stage_samples(cfg_work, hq_, hk_, hv_, max(4, n_rows // 8))}

    qkvo_gb = 4 * q.numel() * 2 / 1e9
    loop = None
    by_config = None
    extra = {}
    del hq_, hk_, hv_, ho, tile_stats, o_full, o_sparse, q, k, v, m, step
    torch.cuda.empty_cache()
    if world == 1 and not args.no_schedule_loop and cfg.total_steps > 1:
        # the workload's real schedule (sustained sparse phase, pattern reuse), same process
        loop = run_schedule_loop(args, cfg, emit=False)
        torch.cuda.empty_cache()
    if world == 1 and not args.no_by_config and cfg.name == "c4":
        # the other workloads, a sharp-logit arm of this one and the paper's short-context setting
        by_config = {}
        for name in ("c2", "c3"):
            by_config[name] = time_config(syn.CONFIGS[name], dev, 20, 3, peaks)
            torch.cuda.empty_cache()
        c5 = syn.CONFIGS["c5"]
        by_config["c5"] = time_config(c5, dev, 10, 3, peaks)
        torch.cuda.empty_cache()
        by_config["c5"]["schedule_loop"] = run_schedule_loop(args, c5, emit=False)
        torch.cuda.empty_cache()
        extra["sharp_logits"] = time_config(cfg.with_(plant_norm=12.0), dev, 5, 2, peaks)
        extra["sharp_logits"]["what"] = ("the headline workload with the planted vectors at norm 12 (logit boost 12.7): "
                                         "sink, stripe and band heads with logit ranges of 10+, where the softmax's "
                                         "rescaling path fires; softmax_rescale_fraction = warp-level rescales per "
                                         "(32 rows x 64 keys) softmax group")
        torch.cuda.empty_cache()
        short = syn.AttnConfig("short32", 8, 32, 32, 4096, 128, 32, 0.5, 2048, seed=32)
        for key, plant in (("short_context_block32", 3.0), ("short_context_block32_sharp", 12.0)):
            extra[key] = time_config(short.with_(plant_norm=plant), dev, 20, 3, peaks)
            extra[key]["what"] = ("the paper's short-context setting: block 32, keep 50 %, L = 4096 (2048 prompt + 2048 "
                                  "generation), batch 8 x 32 heads; TFLOP/s counted on kept-block FLOPs only. Four "
                                  "neighbouring query blocks share an MMA tile and walk the union of their lists: "
                                  "useful_fraction_of_tile_work = sum of list lengths / (4 x union size), 1 when "
                                  "neighbours keep the same blocks (sharp heads), towards 0.5 for independent lists")
            torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": n, "warmup": args.warmup,
        "ms_per_step": total_ms / n, "higher_is_better": True, "scaling": "strong" if shard_heads else "weak",
        "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": bench_config(cfg, k_pre, k_gen, world, shard_heads),
        "pct_bf16_peak": 100.0 * per_gpu_sparse / peak,
        "pct_bf16_peak_sustained": 100.0 * per_gpu_sparse / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None,
        "pct_bf16_nominal_2250": 100.0 * per_gpu_sparse / 2250.0,
        "dense_tflops": dense_tflops, "dense_with_stats_tflops": dense_stats_tflops,
        "speedup_vs_dense": dense_plain_total / sparse_total,
        "speedup_vs_dense_with_stats": full_total / sparse_total, "ideal_speedup": nb / (k_pre + k_gen),
        "phase_ms": {"attn_full_stats": full_total / n, "select_from_stats": select_total / n,
                     "attn_sparse": sparse_total / n, "attn_full_plain (timed after the steps)": dense_plain_total / n},
        "roofline": dominant, "roofline_by_kernel": roof_all,
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "what": "pinned host Q,K,V -> device, sparsed_attn_sparse, O -> pinned host; chunks of 4 kv heads on 3 streams", "steps": e2e_steps,
                "ms_per_step": e2e_ms / e2e_steps},
        "gpu_launches": launches_per_step * n,
        "launches_per_step": {"attn_dense_pair_kernel (dense + row statistics)": 1,
                              "pool_select_kernel (pooling + top-k + CSR)": 1, "attn_kernel<sparse>": 1},
        "clocks": clocks, "peaks": peaks, "schedule_loop": loop, "by_config": by_config,
    }
    line.update(extra)
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_topk_only(args, cfg):
    """The ranking/compaction kernel alone on seeded pseudo scores of this workload's shape
    ([B,Hq,nb,nb] fp32): a small-footprint run for profiling that kernel by itself."""
    import paper_2509_24014_b200 as sd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    peaks = load_peaks()
    B, Hq, nb = cfg.batch, cfg.heads_q, cfg.num_blocks
    scores = syn.random_scores(B * Hq * nb, nb, seed=cfg.seed, device=dev).view(B, Hq, nb, nb)
    params = sd.make_params(cfg.block_size, cfg.keep_ratio, cfg.prefill_len)
    k_pre, k_gen = sd.sparsed_kept_per_row(params, cfg.seq_len)
    pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
    ws = sd.new_workspace(256, dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    times = []
    for _ in range(args.warmup + args.steps):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        sd.sparsed_select_from_scores(scores, params, pat, ws)
        b.record()
        torch.cuda.synchronize()
        times.append(a.elapsed_time(b))
    ms = statistics.median(times[args.warmup:])
    nbytes = B * Hq * (4 * nb * nb + 4 * nb * (k_pre + k_gen) + 4 * nb)
    print(json.dumps({"kernel": "topk_csr_kernel", "workload": workload_name(cfg), "rows": B * Hq * nb, "nb": nb,
                      "ms": ms, "algorithmic_bytes": nbytes, "gbs": nbytes / ms / 1e6,
                      "frac_of_hbm_peak": nbytes / ms / 1e6 / peaks["hbm_gbs"], "l2": "flushed before each launch"}))


def run_schedule_loop(args, cfg, emit=True):
    """The denoising-loop workloads: every step asks the schedule helper for its mode and makes the
    matching library call(s). c4: one layer, 64 steps, fresh noise on Q/K/V each step, pattern selected
    once at the switch step and reused. c5: four layers, 256 steps, the same Q/K/V every step.
    Reports per-phase times, the speedup over all-full attention and (c4) the final-step output error
    against the oracle on sampled rows. Only library calls are inside the timed events; drawing the
    inputs is not."""
    import paper_2509_24014_b200 as sd
    from oracle import sparsed_oracle as orc
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    T, skip, bs = cfg.total_steps, cfg.skip, cfg.block_size
    s_switch = sd.sparsed_switch_step(T, skip)
    B, Hq, L, nb = cfg.batch, cfg.heads_q, cfg.seq_len, cfg.num_blocks
    params = sd.make_params(bs, cfg.keep_ratio, cfg.prefill_len)
    k_pre, k_gen = sd.sparsed_kept_per_row(params, L)
    ws = sd.new_workspace(256, dev)
    layers = []
    for layer in range(cfg.layers):
        base = syn.make_base(cfg, dev, layer) if cfg.step_noise > 0 else None
        qkv = None if base is not None else syn.make_qkv(cfg, dev, layer)
        pat, row_ptr, col_idx = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
        layers.append({"base": base, "qkv": qkv, "pat": pat, "row_ptr": row_ptr, "col_idx": col_idx})
    o = torch.empty(B, Hq, L, cfg.head_dim, dtype=torch.bfloat16, device=dev)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=dev)
    stats = sd.new_tile_stats(o, bs)
    times = {"full": [], "select": [], "sparse": []}
    sample_heads = [0, Hq // 2, Hq - 1]
    sample_blocks = [0, nb // 2 + 1, nb - 1]
    switch_qk = {}
    final = {}
    # warm-up of the three kernels
    q, k, v = layers[0]["qkv"] if layers[0]["qkv"] is not None else syn.make_qkv(cfg, dev, 0, step=0, base=layers[0]["base"])
    for _ in range(2):
        sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, bs)
        sd.sparsed_select_from_stats(q, k, params, lse, stats, layers[0]["pat"], ws)
        sd.sparsed_attn_sparse(q, k, v, o, layers[0]["pat"], ws)
    torch.cuda.synchronize()
    wall0 = time.perf_counter()
    for t in range(1, T + 1):
        mode = sd.sparsed_schedule_mode(t, T, skip)
        for li, lay in enumerate(layers):
            if lay["base"] is not None:
                q, k, v = syn.make_qkv(cfg, dev, li, step=t, base=lay["base"])
            else:
                q, k, v = lay["qkv"]
            a, b, c = _ev(), _ev(), _ev()
            a.record()
            if mode == sd.MODE_FULL:
                sd.sparsed_attn_full(q, k, v, o, None, ws)
                b.record()
                times["full"].append((a, b))
            elif mode == sd.MODE_FULL_AND_SELECT:
                sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, bs)
                b.record()
                sd.sparsed_select_from_stats(q, k, params, lse, stats, lay["pat"], ws)
                c.record()
                times["full"].append((a, b))
                times["select"].append((b, c))
                if cfg.step_noise > 0:
                    for h in sample_heads:
                        switch_qk[h] = (q[0, h].to("cpu"), k[0, h // (Hq // cfg.heads_kv)].to("cpu"))
            else:
                sd.sparsed_attn_sparse(q, k, v, o, lay["pat"], ws)
                b.record()
                times["sparse"].append((a, b))
            if t == T and li == 0 and cfg.step_noise > 0:
                torch.cuda.synchronize()
                for h in sample_heads:
                    hk = h // (Hq // cfg.heads_kv)
                    final[h] = (q[0, h].to("cpu"), k[0, hk].to("cpu"), v[0, hk].to("cpu"), o[0, h].to("cpu"))
    torch.cuda.synchronize()
    wall = time.perf_counter() - wall0
    code, where = sd.sparsed_last_device_status(ws)
    if code != 0:
        raise RuntimeError(f"device status {code} at {where}")
    ms = {kk: [x.elapsed_time(y) for x, y in vv] for kk, vv in times.items()}
    med = {kk: (statistics.median(vv) if vv else None) for kk, vv in ms.items()}
    total = sum(sum(vv) for vv in ms.values())
    n_calls = cfg.layers * T
    out = {"workload": workload_name(cfg) + f", T={T}, skip={skip}, layers={cfg.layers}", "switch_step": s_switch,
           "calls": {kk: len(vv) for kk, vv in ms.items()}, "median_ms": med,
           "total_attention_ms": total, "speedup_sparse_vs_full_step": med["full"] / med["sparse"],
           "ideal_step_speedup": nb / (k_pre + k_gen), "kept_per_row": [k_pre, k_gen],
           "dense_tflops_median": dense_flops(cfg) / med["full"] / 1e9,
           "sparse_tflops_median": sparse_flops(cfg, int(layers[0]["pat"].nnz)) / med["sparse"] / 1e9,
           "wall_s_including_input_generation": wall}
    if args.all_full:
        # the same number of calls with full attention only, timed as one loop
        q, k, v = layers[0]["qkv"] if layers[0]["qkv"] is not None else syn.make_qkv(cfg, dev, 0, step=1, base=layers[0]["base"])
        a, b = _ev(), _ev()
        a.record()
        for _ in range(n_calls):
            sd.sparsed_attn_full(q, k, v, o, None, ws)
        b.record()
        torch.cuda.synchronize()
        out["all_full_attention_ms"] = a.elapsed_time(b)
        out["speedup_whole_schedule_measured"] = out["all_full_attention_ms"] / total
    else:
        out["all_full_attention_ms_estimated"] = n_calls * med["full"]
        out["speedup_whole_schedule_estimated"] = n_calls * med["full"] / total
    n_full = len(ms["full"])
    out["ideal_whole_schedule_speedup"] = n_calls / (n_full + (n_calls - n_full) * (k_pre + k_gen) / nb)
    if final:
        # final-step output error on sampled rows: the oracle attends on the final step's tensors with
        # (a) the GPU's pattern and (b) its own fp64 selection from the switch step's tensors
        f64 = lambda x: x.to(torch.float64).numpy()
        rp, ci = layers[0]["row_ptr"].cpu().numpy(), layers[0]["col_idx"].cpu().numpy()
        pb = cfg.prefill_len // bs
        err_gpu_pat, err_own_pat, same_lists = [], [], []
        for h in sample_heads:
            qh, kh, vh, oh = (f64(x) for x in final[h])
            qs, ks = (f64(x) for x in switch_qk[h])
            for ib in sample_blocks:
                r = h * nb + ib
                gpu_list = list(ci[rp[r]:rp[r + 1]])
                own_list = orc.select_row(orc.head_pooled_row(qs, ks, ib, bs), pb, cfg.keep_ratio)
                rows = slice(ib * bs, (ib + 1) * bs)
                err_gpu_pat.append(np.abs(oh[rows] - orc.head_sparse_rows(qh, kh, vh, ib, gpu_list, bs)).max())
                err_own_pat.append(np.abs(oh[rows] - orc.head_sparse_rows(qh, kh, vh, ib, own_list, bs)).max())
                same_lists.append(gpu_list == own_list)
        out["final_step_max_abs_err_vs_oracle_same_pattern"] = float(max(err_gpu_pat))
        out["final_step_max_abs_err_vs_oracle_own_pattern"] = float(max(err_own_pat))
        out["sampled_rows"] = len(same_lists)
        out["sampled_rows_with_identical_lists"] = int(sum(same_lists))
    if emit:
        print(json.dumps(out))
    return out


def run_sweep(args, cfg):
    """Timed variants of the method on one workload shape (the paper's ablation axes, latency only):
    keep ratio, isolated vs plain selection, re-selecting every step, no full-attention prefix, and
    the sliding-window / sink+window comparison patterns through the same sparse kernel."""
    import paper_2509_24014_b200 as sd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    q, k, v = syn.make_qkv(cfg, dev)
    B, Hq, L, D = q.shape
    bs, nb = cfg.block_size, cfg.num_blocks
    o = torch.empty_like(q)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=dev)
    stats = sd.new_tile_stats(q, bs)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_PATTERN, sd.make_shape(q, k),
                                                      sd.make_params(bs, cfg.keep_ratio, cfg.prefill_len)), dev)

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = _ev(), _ev()
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    full_ms = timed(lambda: sd.sparsed_attn_full(q, k, v, o, None, ws), reps=3)
    full_stats_ms = timed(lambda: sd.sparsed_attn_full_stats(q, k, v, o, lse, stats, ws, bs), reps=3)
    rows = []
    for rho in (0.05, 0.1, 0.2, 0.3, 0.5):
        for p_len in sorted({0, cfg.prefill_len, L // 2}):
            params = sd.make_params(bs, rho, p_len)
            k_pre, k_gen = sd.sparsed_kept_per_row(params, L)
            pat, rp, ci = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
            sel_ms = timed(lambda: sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws))
            sp_ms = timed(lambda: sd.sparsed_attn_sparse(q, k, v, o, pat, ws))
            rows.append({"keep_ratio": rho, "prefill_len": p_len, "kept_per_row": [k_pre, k_gen],
                         "select_from_stats_ms": sel_ms, "sparse_ms": sp_ms,
                         "sparse_tflops": sparse_flops(cfg, int(pat.nnz)) / sp_ms / 1e9,
                         "speedup_vs_full": full_ms / sp_ms, "ideal": nb / (k_pre + k_gen)})
    # the paper's ablation rows as per-step attention time at this shape
    params = sd.make_params(bs, cfg.keep_ratio, cfg.prefill_len)
    k_pre, k_gen = sd.sparsed_kept_per_row(params, L)
    pat, rp, ci = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
    sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws)
    sp_ms = timed(lambda: sd.sparsed_attn_sparse(q, k, v, o, pat, ws))
    resel_ms = timed(lambda: sd.sparsed_select_pattern(q, k, params, pat, ws, lse=None), reps=3)
    T, skip = (cfg.total_steps, cfg.skip) if cfg.total_steps > 1 else (64, 0.2)   # workloads without a schedule: the 64k one's
    s_sw = sd.sparsed_switch_step(T, skip)
    sel_ms = timed(lambda: sd.sparsed_select_from_stats(q, k, params, lse, stats, pat, ws))
    total_sparsed = (s_sw - 1) * full_ms + full_stats_ms + sel_ms + (T - s_sw) * sp_ms
    ablation = {
        "T": T, "skip": skip, "switch_step": s_sw, "full_step_ms": full_ms, "sparse_step_ms": sp_ms,
        "all_full_ms": T * full_ms, "sparsed_ms": total_sparsed,
        "no_skipping_ms (skip=0: select at step 1)": full_stats_ms + sel_ms + (T - 1) * sp_ms,
        "no_reuse_ms (re-select every sparse step, own QK^T pass incl. row statistics)":
            (s_sw - 1) * full_ms + full_stats_ms + sel_ms + (T - s_sw) * (resel_ms + sp_ms),
        "reselect_ms": resel_ms,
    }
    # comparison patterns: sliding window ws = l/2 and sink (10 % of the keys) + window
    base = {}
    for name, sink, window in (("sliding_window_ws_l/2", 0, nb // 2 + 1), ("sink10%+window_ws_l/2", max(1, nb // 10), nb // 2 + 1)):
        wpat, wrp, wci = sd.sparsed_build_window_pattern(B, Hq, nb, bs, sink, window, dev)
        w_ms = timed(lambda: sd.sparsed_attn_sparse(q, k, v, o, wpat, ws))
        base[name] = {"nnz": int(wpat.nnz), "density": int(wpat.nnz) / (B * Hq * nb * nb), "sparse_ms": w_ms,
                      "sparse_tflops": sparse_flops(cfg, int(wpat.nnz)) / w_ms / 1e9, "speedup_vs_full": full_ms / w_ms}
    print(json.dumps({"workload": workload_name(cfg), "full_ms": full_ms, "full_with_stats_ms": full_stats_ms,
                      "dense_tflops": dense_flops(cfg) / full_ms / 1e9, "keep_ratio_sweep": rows,
                      "ablation_schedule_ms": ablation, "comparison_patterns": base}))


def run_estimate_recall(args, cfg):
    """The exact switch-step selection beside the block-mean estimate (pool Q and K first, then score; not the
    paper's scorer) on the same inputs: time of each, how much of the exact pattern the estimate recovers
    (by count and by A' mass) and the error each pattern leaves in the sparse output against full attention,
    per planted head kind."""
    import numpy as np
    import paper_2509_24014_b200 as sd
    from paper_2509_24014_b200 import pattern_metrics as pm
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    q, k, v = syn.make_qkv(cfg, dev)
    B, Hq, L, D = q.shape
    bs, nb = cfg.block_size, cfg.num_blocks
    params = sd.make_params(bs, cfg.keep_ratio, cfg.prefill_len)
    k_pre, k_gen = sd.sparsed_kept_per_row(params, L)
    o_full, o_sp = torch.empty_like(q), torch.empty_like(q)
    lse = torch.empty(B, Hq, L, dtype=torch.float32, device=dev)
    stats = sd.new_tile_stats(q, bs)
    ws = sd.new_workspace(sd.sparsed_workspace_bytes(sd.OP_SELECT_POOLED_QK, sd.make_shape(q, k), params), dev)
    scores = torch.empty(B, Hq, nb, nb, dtype=torch.float32, device=dev)
    pat_x, rp_x, ci_x = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)
    pat_e, rp_e, ci_e = sd.new_pattern(B, Hq, nb, k_pre + k_gen, dev)

    def timed(fn, reps=5):
        fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(reps):
            a, b = _ev(), _ev()
            a.record(); fn(); b.record()
            torch.cuda.synchronize()
            ts.append(a.elapsed_time(b))
        return statistics.median(ts)

    sd.sparsed_attn_full_stats(q, k, v, o_full, lse, stats, ws, bs)
    exact_ms = timed(lambda: sd.sparsed_select_from_stats(q, k, params, lse, stats, pat_x, ws, scores_out=scores))
    est_ms = timed(lambda: sd.sparsed_select_pattern_pooled_qk(q, k, params, pat_e, ws))
    torch.cuda.synchronize()
    a_exact = scores.cpu().numpy().reshape(B * Hq * nb, nb)
    rpx, cix, rpe, cie = (t.cpu().numpy() for t in (rp_x, ci_x, rp_e, ci_e))
    recall = pm.pattern_recall(rpx, cix, rpe, cie, nb).reshape(B, Hq, nb)
    mass_x = pm.kept_mass(a_exact, rpx, cix).reshape(B, Hq, nb) * bs     # share of each row block's probability mass
    mass_e = pm.kept_mass(a_exact, rpe, cie).reshape(B, Hq, nb) * bs

    def out_err(pat):
        sd.sparsed_attn_sparse(q, k, v, o_sp, pat, ws)
        torch.cuda.synchronize()
        num = torch.stack([(o_sp[:, h].float() - o_full[:, h].float()).norm() for h in range(Hq)])
        den = torch.stack([o_full[:, h].float().norm() for h in range(Hq)])
        return (num / den).cpu().numpy()

    err_x, err_e = out_err(pat_x), out_err(pat_e)
    assert sd.sparsed_last_device_status(ws) == (0, 0)
    kinds = [kd[0] for kd in syn.head_kinds(cfg)]
    by_kind = {}
    for name in sorted(set(kinds)):
        hs = [h for h in range(Hq) if kinds[h] == name]
        by_kind[name] = {"heads": len(hs), "recall": float(recall[:, hs].mean()),
                         "kept_mass_exact": float(mass_x[:, hs].mean()), "kept_mass_estimate": float(mass_e[:, hs].mean()),
                         "sparse_vs_full_rel_err_exact": float(err_x[hs].mean()),
                         "sparse_vs_full_rel_err_estimate": float(err_e[hs].mean())}
    print(json.dumps({"workload": workload_name(cfg), "plant_norm": cfg.plant_norm,
                      "select_from_stats_ms": exact_ms, "select_pooled_qk_ms": est_ms,
                      "recall_of_exact_pattern": float(recall.mean()), "kept_mass_exact": float(mass_x.mean()),
                      "kept_mass_estimate": float(mass_e.mean()), "sparse_vs_full_rel_err_exact": float(err_x.mean()),
                      "sparse_vs_full_rel_err_estimate": float(err_e.mean()), "by_head_kind": by_kind}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c4", choices=sorted(syn.CONFIGS))
    ap.add_argument("--cpu-rows", type=int, default=128, help="row blocks the CPU oracle is timed on")
    ap.add_argument("--ref-rows", type=int, default=12, help="row blocks per step of the reference arm")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--only-topk", action="store_true", help="run only the stand-alone ranking kernel")
    ap.add_argument("--schedule-loop", action="store_true",
                    help="run the config's whole denoising schedule (c4: 64 steps, c5: 4 layers x 256 steps)")
    ap.add_argument("--all-full", action="store_true", help="with --schedule-loop: also time all-full attention")
    ap.add_argument("--no-schedule-loop", action="store_true", help="skip the schedule-loop summary of the default run")
    ap.add_argument("--no-by-config", action="store_true",
                    help="skip the summary of the other workloads (c2, c3, c5, sharp logits, block 32)")
    ap.add_argument("--shard", default="replicas", choices=["replicas", "heads"],
                    help="with --gpus N > 1: independent replicas (default) or one layer's heads split over the ranks")
    ap.add_argument("--sweep", action="store_true", help="keep-ratio / isolation / ablation / comparison-pattern timings")
    ap.add_argument("--estimate-recall", action="store_true",
                    help="exact selection vs the block-mean estimate: time, recall, kept mass, output error")
    ap.add_argument("--plant-norm", type=float, default=None,
                    help="norm of the planted vectors (default 3: logit boost 0.8; 9 gives sharp attention)")
    args = ap.parse_args()
    cfg = syn.CONFIGS[args.config]
    if args.plant_norm is not None:
        cfg = cfg.with_(plant_norm=args.plant_norm)
    if args.estimate_recall:
        run_estimate_recall(args, cfg)
    elif args.sweep:
        run_sweep(args, cfg)
    elif args.schedule_loop:
        run_schedule_loop(args, cfg)
    elif args.only_topk:
        run_topk_only(args, cfg)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
