#!/usr/bin/env python
"""Benchmark of the PowerAttention hot path on B200: prints ONE JSON line.

A step is one pass of the whole path on resident synthetic inputs: pa_build_layout +
pa_prefill at 128K tokens (28 query / 4 KV heads, head_dim 128, block 64, window 5, sink 1)
followed by pa_decode on the batch-8 decode workload.  The metric is the prefill's active-block
throughput: 4 * 64 * 64 * head_dim FLOP per listed block pair per query head, over the step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1 (under torchrun) runs independent replicas, one per GPU: the operator has no exchange
step, so there is no collective on the data path; time is the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import synth_inputs as si  # noqa: E402

METRIC = "prefill_active_block_tflops_128k"
UNIT = "TFLOP/s"


def block_pair_flops(nnz: int, w) -> float:
    return 4.0 * w.block * w.block * w.head_dim * nnz * w.n_q_heads * w.batch


def read_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# DRAM bytes moved by one prefill_kernel<128> launch on the 128K workload: dram__bytes_read.sum +
# dram__bytes_write.sum of an ncu capture of this very workload.  The figure belongs to the kernel
# sources it was taken on: once they change it is reported as null until the capture is repeated.
PREFILL_TRAFFIC = dict(
    bytes=1640398336 + 913427712,
    sources={
        "prefill_sm100.cu": "1cb4861353d25e54a2b0827487fb7dac9e2be1f551e31ca3d82349e8868b803c",
        "sm100_ptx.cuh": "f0dd47ba76fa3fd147120ccffa5c14e4d442cb67ae25aedcff0959f1dbb6ad64",
    },
)


def prefill_traffic():
    import hashlib

    csrc = os.path.join(ROOT, "paper_2503_03588_b200", "csrc")
    for name, digest in PREFILL_TRAFFIC["sources"].items():
        try:
            with open(os.path.join(csrc, name), "rb") as f:
                if hashlib.sha256(f.read()).hexdigest() != digest:
                    return None
        except OSError:
            return None
    return PREFILL_TRAFFIC["bytes"]


# ------------------------------------------------------------------------------ multi-rank glue

def dist_env():
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return world, rank, local


def aggregate(ms_local: float, flops_local: float, group=None, device="cpu"):
    """Replica aggregation: job time = max over ranks, job work = sum over ranks."""
    import torch.distributed as dist

    if not (dist.is_available() and dist.is_initialized()):
        return ms_local, flops_local
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    f = torch.tensor([flops_local], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX, group=group)
    dist.all_reduce(f, op=dist.ReduceOp.SUM, group=group)
    return float(t.item()), float(f.item())


# ------------------------------------------------------------------------------ clocks

class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu), "-lms", "20"], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            # The timed region is a few tens of milliseconds: return only once the sampler is
            # producing lines, so that it is known to run while the steps are timed.
            t0 = time.time()
            while time.time() - t0 < 3.0 and os.path.getsize(self.path) == 0:
                time.sleep(0.01)
            self.first_bytes = os.path.getsize(self.path)
        except Exception:
            self.proc = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[])
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            with open(self.path) as fh:
                idle = fh.read(getattr(self, "first_bytes", 0)).splitlines()  # taken before start() returned
                lines = fh.readlines() or idle[-1:]
            for line in lines:
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                sm.append(float(f[1]))
                smax.append(float(f[2]))
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out = dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(smax)), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ------------------------------------------------------------------------------ reference arm

def oracle_sample_rows(w, every: int):
    """Every `every`-th query block of the workload, all 64 rows of each."""
    nqb = w.seq_len // w.block
    blocks = np.arange(nqb - 1, -1, -every)
    return np.sort((blocks[:, None] * w.block + np.arange(w.block)[None, :]).reshape(-1))


def time_oracle(w, Q, K, V, every: int, nnz_rows_flops, keep=None):
    """Times the fp64 oracle, as it stands, on the sampled rows; returns (seconds, flops, cores, rows).
    `keep`, a dict, receives the rows and the oracle's results for a comparison with the GPU's."""
    from oracle import oracle

    rows = oracle_sample_rows(w, every)
    t0 = time.time()
    o_ref, lse_ref, _ = oracle.prefill(Q, K, V, w.block, w.window_blocks, w.sink_blocks, rows=rows)
    dt = time.time() - t0
    if keep is not None:
        keep.update(rows=rows, o=o_ref, lse=lse_ref)
    return dt, nnz_rows_flops(rows), oracle.max_threads(), len(rows)


def run_reference(args):
    world, rank, _ = dist_env()
    if rank != 0:
        return
    from oracle import oracle

    w = si.PREFILL_128K
    Q, K, V = si.prefill_inputs(w)
    rp, _ = oracle.block_layout(w.seq_len, w.block, w.window_blocks, w.sink_blocks)
    row_len = np.diff(rp)

    def flops_of(rows):
        blocks = np.unique(rows // w.block)
        return 4.0 * w.block * w.block * w.head_dim * float(row_len[blocks].sum()) * w.n_q_heads

    every = 64  # 32 query blocks = 2048 rows per step: a few seconds of CPU work
    times = []
    for it in range(args.warmup + args.steps):
        dt, fl, cores, nrows = time_oracle(w, Q, K, V, every, flops_of)
        if it >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    value = fl / (ms * 1e-3) / 1e12
    sample = f"every {every}th query block of the 128K workload ({nrows} rows, all 28 heads) per step"
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=ms, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=w.name, seq_len=w.seq_len, n_q_heads=w.n_q_heads,
                            n_kv_heads=w.n_kv_heads, head_dim=w.head_dim, block=w.block,
                            window_blocks=w.window_blocks, sink_blocks=w.sink_blocks),
                cpu_baseline=dict(value=value, unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line))


# ------------------------------------------------------------------------------ our arm

def run_ours(args):
    import paper_2503_03588_b200 as pa  # raises if the CUDA library is missing: no fallback

    world, rank, local = dist_env()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (B200)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    peaks = read_peaks()

    w, wd = si.PREFILL_128K, si.DECODE_B8
    Qh, Kh, Vh = si.prefill_inputs(w, pin=True)
    nqb, nnz = pa.pa_layout_size(w.seq_len, w.block, w.window_blocks, w.sink_blocks)
    flops = block_pair_flops(nnz, w)
    n_heads_local = w.n_q_heads
    if args.shard_heads and world > 1:
        # Strong scaling without an exchange step: each rank takes whole KV heads and their query
        # heads of the same problem (at most n_kv_heads ranks have work; an idle rank repeats rank
        # 0's first group, uncounted).
        from paper_2503_03588_b200.sharding import kv_head_shard

        qs, ks = kv_head_shard(w.n_q_heads, w.n_kv_heads, world, rank)
        if ks.start == ks.stop:
            qs, ks, flops = slice(0, w.n_q_heads // w.n_kv_heads), slice(0, 1), 0.0
        Qh, Kh, Vh = (t.contiguous().pin_memory() for t in (Qh[:, :, qs], Kh[:, :, ks], Vh[:, :, ks]))
        n_heads_local = qs.stop - qs.start
        if flops:
            flops *= n_heads_local / w.n_q_heads
    Q, K, V = Qh.to(dev), Kh.to(dev), Vh.to(dev)
    row_ptr = torch.empty(nqb + 1, dtype=torch.int32, device=dev)
    col_idx = torch.empty(nnz, dtype=torch.int32, device=dev)
    O = torch.empty_like(Q)
    LSE = torch.empty((w.batch, n_heads_local, w.seq_len), dtype=torch.float32, device=dev)
    ws = torch.empty(4096, dtype=torch.uint8, device=dev)

    qd_h, kc_h, vc_h, lens = si.decode_inputs(wd)
    qd, kc, vc = qd_h.to(dev), kc_h.to(dev), vc_h.to(dev)
    del kc_h, vc_h
    lens_d = torch.as_tensor(lens, dtype=torch.int32, device=dev)
    Od = torch.empty((wd.batch, wd.n_q_heads, wd.head_dim), dtype=torch.bfloat16, device=dev)
    LSEd = torch.empty((wd.batch, wd.n_q_heads), dtype=torch.float32, device=dev)
    dparams = pa.binding.decode_params(qd, kc, vc, wd.window_blocks, wd.sink_blocks)
    wsd = torch.empty(pa.pa_decode_workspace_bytes(dparams), dtype=torch.uint8, device=dev)

    stream = torch.cuda.current_stream()
    ev_p0 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ev_p1 = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]

    def step(i=None):
        pa.pa_build_layout(w.seq_len, w.block, w.window_blocks, w.sink_blocks, row_ptr, col_idx)
        if i is not None:
            ev_p0[i].record(stream)
        pa.pa_prefill(Q, K, V, row_ptr, col_idx, o=O, lse=LSE, workspace=ws)
        if i is not None:
            ev_p1[i].record(stream)
        pa.pa_decode(qd, kc, vc, lens_d, wd.window_blocks, wd.sink_blocks, o=Od, lse=LSEd, workspace=wsd)

    launches_per_step = 3 + 1 + 1  # layout (count, scan, fill) + prefill + decode (one cluster kernel)

    for _ in range(max(args.warmup, 3)):
        step()
    pa.pa_prefill_status(ws)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(args.steps):
        step(i)
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        torch.distributed.barrier()
    pa.pa_prefill_status(ws)
    ms_local = e0.elapsed_time(e1) / args.steps
    prefill_ms = float(np.mean([a.elapsed_time(b) for a, b in zip(ev_p0, ev_p1)]))
    ms, flops_all = aggregate(ms_local, flops, device=dev)

    if rank != 0:
        if world > 1:
            torch.distributed.destroy_process_group()
        return

    # ---- decode bandwidth: CUDA graph of launches rotating over 16 seeded length sets so that
    # consecutive launches touch different cache regions (touched bytes per call fit in L2).
    n_sets, reps = 16, 8
    rng = np.random.Generator(np.random.PCG64(wd.lens_seed + 1))
    lens_sets = [rng.integers(wd.min_len, wd.max_len + 1, size=wd.batch, dtype=np.int64) for _ in range(n_sets)]
    lens_sets_d = [torch.as_tensor(x, dtype=torch.int32, device=dev) for x in lens_sets]

    def touched_bytes(ls):
        total = 0
        for L in ls:
            nblk = len(pa.pa_decode_block_list(int(L), wd.block, wd.window_blocks, wd.sink_blocks))
            keys = wd.block * (nblk - 1) + (int(L) - 1) % wd.block + 1
            total += keys * wd.head_dim * 2 * 2 * wd.n_kv_heads
        return total

    dec_bytes = float(np.mean([touched_bytes(ls) for ls in lens_sets]))
    side = torch.cuda.Stream(device=dev)
    side.wait_stream(stream)
    with torch.cuda.stream(side):
        for ld in lens_sets_d:
            pa.pa_decode(qd, kc, vc, ld, wd.window_blocks, wd.sink_blocks, o=Od, lse=LSEd, workspace=wsd)
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for _ in range(reps):
                for ld in lens_sets_d:
                    pa.pa_decode(qd, kc, vc, ld, wd.window_blocks, wd.sink_blocks, o=Od, lse=LSEd, workspace=wsd)
        graph.replay()
        torch.cuda.synchronize()
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        d0.record(side)
        graph.replay()
        d1.record(side)
        torch.cuda.synchronize()
    dec_us = 1e3 * d0.elapsed_time(d1) / (n_sets * reps)
    dec_gbs = dec_bytes / (dec_us * 1e-6) / 1e9

    # ---- what a kernel launch costs in such a graph: 128 launches of a one-element library kernel,
    # timed the same way (the decode call's time is several of these, so launch latency is not its floor).
    tiny = torch.zeros(1, device=dev)
    with torch.cuda.stream(side):
        tiny.add_(1.0)
        torch.cuda.synchronize()
        gf = torch.cuda.CUDAGraph()
        with torch.cuda.graph(gf, stream=side):
            for _ in range(n_sets * reps):
                tiny.add_(1.0)
        gf.replay()
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record(side)
        gf.replay()
        f1.record(side)
        torch.cuda.synchronize()
    floor_us = 1e3 * f0.elapsed_time(f1) / (n_sets * reps)

    # ---- the same calls issued eagerly (no graph): device time per call and the host's time to
    # enqueue one (argument checks, cached tensor maps, the launch), which a graph replay hides.
    def eager(fn, n):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        g0.record(stream)
        for _ in range(n):
            fn()
        g1.record(stream)
        host_us = 1e6 * (time.perf_counter() - t0) / n
        torch.cuda.synchronize()
        return dict(device_us_per_call=1e3 * g0.elapsed_time(g1) / n, host_enqueue_us_per_call=host_us, calls=n)

    it = iter(range(1 << 30))
    eager_decode = eager(lambda: pa.pa_decode(qd, kc, vc, lens_sets_d[next(it) % n_sets], wd.window_blocks, wd.sink_blocks,
                                              o=Od, lse=LSEd, workspace=wsd), 256)
    eager_prefill = eager(lambda: pa.pa_prefill(Q, K, V, row_ptr, col_idx, o=O, lse=LSE, workspace=ws), 10)

    # ---- many decoding steps against a paged cache (the paper's serving shape: a long input, then
    # 1024 decoding steps): batch 8 at 16K tokens, every step appends one token's K and V and
    # decodes.  128 steps are captured in a graph (the lengths live on the device and advance by
    # themselves) and replayed eight times.
    def decode_steps():
        ctx, steps, per_graph = 16384, 1024, 128
        max_blocks = (ctx + steps + 63) // 64
        n_pages = wd.batch * max_blocks
        gen = torch.Generator(device=dev)
        gen.manual_seed(wd.seed + 7)
        shape = (n_pages, 64, wd.n_kv_heads, wd.head_dim)
        kp = torch.randn(shape, device=dev, dtype=torch.bfloat16, generator=gen)
        vp = torch.randn(shape, device=dev, dtype=torch.bfloat16, generator=gen)
        perm = torch.randperm(n_pages, device=dev, generator=gen).to(torch.int32)
        table = perm.view(wd.batch, max_blocks).contiguous()
        lens_s = torch.full((wd.batch,), ctx, dtype=torch.int32, device=dev)
        k_new = torch.randn((wd.batch, wd.n_kv_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
        v_new = torch.randn_like(k_new)
        o_s, lse_s, ws_s = pa.pa_decode_paged(qd, kp, vp, table, lens_s, wd.window_blocks, wd.sink_blocks)

        def one_step():
            pa.pa_kv_append(k_new, v_new, kp, vp, table, lens_s)
            pa.pa_decode_paged(qd, kp, vp, table, lens_s, wd.window_blocks, wd.sink_blocks, o=o_s, lse=lse_s, workspace=ws_s)

        with torch.cuda.stream(side):
            one_step()
            torch.cuda.synchronize()
            lens_s.fill_(ctx)
            gs = torch.cuda.CUDAGraph()
            with torch.cuda.graph(gs, stream=side):
                for _ in range(per_graph):
                    one_step()
            torch.cuda.synchronize()
            lens_s.fill_(ctx)
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            s0.record(side)
            for _ in range(steps // per_graph):
                gs.replay()
            s1.record(side)
            torch.cuda.synchronize()
        assert int(lens_s[0].item()) == ctx + steps
        pa.pa_decode_status(ws_s)
        return dict(workload="batch 8, 16K-token context + 1024 steps, paged cache (64-token pages), append + decode per step",
                    us_per_step=1e3 * s0.elapsed_time(s1) / steps, steps=steps, launches_per_step=3)

    decode_many = decode_steps()

    # ---- the 32K prefill workload (the metric is quoted at 32K and 128K): same kernel, K scaled so
    # that the logits have a standard deviation of about 3; its inputs (0.6 GB) exceed L2.
    w32 = si.PREFILL_32K
    Q32, K32, V32 = (t.to(dev) for t in si.prefill_inputs(w32))
    rp32, ci32 = pa.pa_build_layout(w32.seq_len, w32.block, w32.window_blocks, w32.sink_blocks)
    o32, lse32, ws32 = pa.pa_prefill(Q32, K32, V32, rp32, ci32)
    for _ in range(3):
        pa.pa_prefill(Q32, K32, V32, rp32, ci32, o=o32, lse=lse32, workspace=ws32)
    torch.cuda.synchronize()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    n32 = 20
    p0.record(stream)
    for _ in range(n32):
        pa.pa_prefill(Q32, K32, V32, rp32, ci32, o=o32, lse=lse32, workspace=ws32)
    p1.record(stream)
    torch.cuda.synchronize()
    pa.pa_prefill_status(ws32)
    ms32 = p0.elapsed_time(p1) / n32
    flops32 = 4.0 * w32.block * w32.block * w32.head_dim * float(ci32.numel()) * w32.n_q_heads * w32.batch
    prefill_32k = dict(workload=w32.name, active_block_pairs=int(ci32.numel()), ms=ms32,
                       value=flops32 / (ms32 * 1e-3) / 1e12, unit=UNIT,
                       frac=flops32 / (ms32 * 1e-3) / 1e12 / peaks["bf16_tflops"], launches=n32)
    # ---- the backward pass on the same 32K workload (dO drawn on the device; values do not matter
    # for time): 10 * 64 * 64 * head_dim FLOP per listed block pair and query head (five products).
    gen32 = torch.Generator(device=dev)
    gen32.manual_seed(w32.seed + 9)
    dO32 = torch.randn(o32.shape, device=dev, dtype=torch.bfloat16, generator=gen32)
    dq32, dk32, dv32, wsb32 = pa.pa_prefill_backward(Q32, K32, V32, o32, lse32, dO32, rp32, ci32)
    torch.cuda.synchronize()
    b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    nb = 5
    b0.record(stream)
    for _ in range(nb):
        pa.pa_prefill_backward(Q32, K32, V32, o32, lse32, dO32, rp32, ci32, dq=dq32, dk=dk32, dv=dv32, workspace=wsb32)
    b1.record(stream)
    torch.cuda.synchronize()
    msb = b0.elapsed_time(b1) / nb
    backward_32k = dict(workload=w32.name, ms=msb, value=2.5 * flops32 / (msb * 1e-3) / 1e12, unit=UNIT,
                        frac=2.5 * flops32 / (msb * 1e-3) / 1e12 / peaks["bf16_tflops"], bound="tensor",
                        flops_per_pair_head=10 * w32.block * w32.block * w32.head_dim, launches=nb,
                        kernels="delta, transposed layout (4), dQ and dK/dV on tcgen05 with accumulators in tensor memory, "
                                "fp32 outputs")
    pa.pa_prefill_status(wsb32)
    del Q32, K32, V32, o32, lse32, dO32, dq32, dk32, dv32

    # ---- decode scale-up (labelled, beside the batch-8 figure): the same per-sequence pattern at
    # larger batches, where one call moves enough bytes to outlast its launch.  Caches are drawn on
    # the device (values do not matter for bandwidth); lengths are seeded like the batch-8 sets.
    scale_up = []
    if not args.no_decode_scale_up:
        for big in (64, 256):
            cache_bytes = 2 * big * wd.max_len * wd.n_kv_heads * wd.head_dim * 2
            if torch.cuda.mem_get_info(dev)[0] < cache_bytes + (8 << 30):
                continue
            gen = torch.Generator(device=dev)
            gen.manual_seed(wd.seed + big)
            kcb = torch.randn((big, wd.max_len, wd.n_kv_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
            vcb = torch.randn((big, wd.max_len, wd.n_kv_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
            qb = torch.randn((big, wd.n_q_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
            rngb = np.random.Generator(np.random.PCG64(wd.lens_seed + big))
            sets_b = [rngb.integers(wd.min_len, wd.max_len + 1, size=big, dtype=np.int64) for _ in range(4)]
            sets_bd = [torch.as_tensor(x, dtype=torch.int32, device=dev) for x in sets_b]
            bytes_b = float(np.mean([touched_bytes(ls) for ls in sets_b]))
            ob, lb, wsb = pa.pa_decode(qb, kcb, vcb, sets_bd[0], wd.window_blocks, wd.sink_blocks)
            with torch.cuda.stream(side):
                torch.cuda.synchronize()
                gb = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gb, stream=side):
                    for _ in range(4):
                        for ld in sets_bd:
                            pa.pa_decode(qb, kcb, vcb, ld, wd.window_blocks, wd.sink_blocks, o=ob, lse=lb, workspace=wsb)
                gb.replay()
                torch.cuda.synchronize()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                g0.record(side)
                gb.replay()
                g1.record(side)
                torch.cuda.synchronize()
            us_b = 1e3 * g0.elapsed_time(g1) / 16
            scale_up.append(dict(batch=big, us_per_call=us_b, kv_bytes_per_call=bytes_b,
                                 value=bytes_b / (us_b * 1e-6) / 1e9, unit="GB/s",
                                 frac=bytes_b / (us_b * 1e-6) / 1e9 / peaks["hbm_gbs"]))
            del kcb, vcb, qb, ob, lb, wsb, gb
            torch.cuda.empty_cache()

    # ---- end to end through the public API with host buffers: pinned H2D of Q, K, V, the call,
    # D2H of O and LSE, all inside the timed region.  Consecutive steps overlap as a serving loop
    # would run them: the copies in of step i+1 and the copies out of step i-1 travel while step i
    # computes (three streams, two sets of device tensors).
    Oh = torch.empty(O.shape, dtype=O.dtype, pin_memory=True)
    LSEh = torch.empty(LSE.shape, dtype=LSE.dtype, pin_memory=True)
    e2e_steps = max(2, min(args.steps, 6))
    sets = [(Q, K, V, O, LSE), tuple(torch.empty_like(t) for t in (Q, K, V, O, LSE))]
    s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    ev_in = [torch.cuda.Event() for _ in range(2)]
    ev_cmp = [torch.cuda.Event() for _ in range(2)]
    ev_out = [torch.cuda.Event() for _ in range(2)]

    def e2e_run(n):
        for i in range(n):
            b = i & 1
            Qd, Kd, Vd, Od, Ld = sets[b]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_cmp[b])  # step i-2 has read this set
                Qd.copy_(Qh, non_blocking=True)
                Kd.copy_(Kh, non_blocking=True)
                Vd.copy_(Vh, non_blocking=True)
                ev_in[b].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in[b])
                if i >= 2:
                    s_cmp.wait_event(ev_out[b])  # step i-2's results have left this set
                pa.pa_build_layout(w.seq_len, w.block, w.window_blocks, w.sink_blocks, row_ptr, col_idx)
                pa.pa_prefill(Qd, Kd, Vd, row_ptr, col_idx, o=Od, lse=Ld, workspace=ws)
                ev_cmp[b].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[b])
                Oh.copy_(Od, non_blocking=True)
                LSEh.copy_(Ld, non_blocking=True)
                ev_out[b].record(s_out)

    e2e_run(2)
    torch.cuda.synchronize()
    x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    x0.record(s_in)
    e2e_run(e2e_steps)
    x1.record(s_out)
    torch.cuda.synchronize()
    pa.pa_prefill_status(ws)
    e2e_ms = x0.elapsed_time(x1) / e2e_steps
    h2d = sum(t.numel() * t.element_size() for t in (Qh, Kh, Vh))
    d2h = sum(t.numel() * t.element_size() for t in (Oh, LSEh))

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample of the same workload.
    cpu = parity = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import oracle

        rp_ref, _ = oracle.block_layout(w.seq_len, w.block, w.window_blocks, w.sink_blocks)
        row_len = np.diff(rp_ref)

        def flops_of(rows):
            blocks = np.unique(rows // w.block)
            return 4.0 * w.block * w.block * w.head_dim * float(row_len[blocks].sum()) * w.n_q_heads

        every = 16
        ref = {}
        dt, fl, cores, nrows = time_oracle(w, Qh, Kh, Vh, every, flops_of, keep=ref)
        cpu = dict(value=fl / dt / 1e12, unit=UNIT, cores=cores, kind="oracle",
                   sample=f"every {every}th query block of the 128K workload ({nrows} rows, all heads), {dt:.1f} s")
        # The rows the oracle has just evaluated, against the GPU's output of the same workload.
        pa.pa_prefill(Q, K, V, row_ptr, col_idx, o=O, lse=LSE, workspace=ws)
        pa.pa_prefill_status(ws)
        ridx = torch.as_tensor(ref["rows"], device=dev)
        eo = np.abs(O[:, ridx].double().cpu().numpy() - ref["o"])
        el = np.abs(LSE[:, :, ridx].double().cpu().numpy() - ref["lse"])
        parity = dict(rows=int(nrows), heads=w.n_q_heads, o_max_abs=float(eo.max()), o_mean_abs=float(eo.mean()),
                      lse_max_abs=float(el.max()), bounds=dict(o_max_abs=2e-2, o_mean_abs=2e-3, lse_max_abs=1e-3),
                      against="fp64 oracle on the cpu_baseline sample")
        del ref

    value = flops_all / (ms * 1e-3) / 1e12
    achieved = flops / (prefill_ms * 1e-3) / 1e12
    # Which measured bf16 peak the kernel is held against: the burst figure while the timed region
    # ran at full clocks (a short run), the sustained one once the median SM clock sampled during it
    # is more than 8 % below the maximum (a long run of a kernel that draws the full board power).  Both fractions
    # are in the line.
    capped = clocks.get("sm_mhz") is not None and clocks["sm_mhz"] < 0.92 * clocks["sm_max_mhz"]
    peak = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
    peak_kind = " sustained bf16 (power-capped clocks in the timed region)" if capped else " burst bf16"
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                ms_per_step=ms, higher_is_better=True,
                scaling="strong" if (args.shard_heads and world > 1) else "weak", vs_baseline=None, dtype="bf16",
                data="synthetic",
                config=dict(workload=w.name, seq_len=w.seq_len, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                            head_dim=w.head_dim, block=w.block, window_blocks=w.window_blocks,
                            sink_blocks=w.sink_blocks, active_block_pairs=nnz, step="layout+prefill+decode",
                            decode_workload=wd.name, l2="inputs larger than L2 (Q+K+V+O = 2.4 GB per step)",
                            parallelism=("kv_head_shards" if args.shard_heads else "replicas") if world > 1 else "single"),
                clocks=clocks,
                roofline=dict(bound="tensor", achieved=achieved, peak=peak, unit="TFLOP/s",
                              frac=achieved / peak, traffic=prefill_traffic(),
                              peak_source=peaks["source"] + peak_kind, kernel="prefill_kernel<128>",
                              kernel_ms=prefill_ms,
                              frac_of_burst=achieved / peaks["bf16_tflops"],
                              frac_of_sustained=achieved / peaks["bf16_tflops_sustained"]),
                prefill_32k=prefill_32k, backward_32k=backward_32k,
                decode=dict(metric="decode_kv_gbs", value=dec_gbs, unit="GB/s", us_per_call=dec_us,
                            kv_bytes_per_call=dec_bytes, peak=peaks["hbm_gbs"], frac=dec_gbs / peaks["hbm_gbs"],
                            launch_floor_us=floor_us,
                            bound="hbm", timing=f"CUDA graph of {n_sets * reps} calls rotating over {n_sets} seeded length sets",
                            workload=wd.name, scale_up=scale_up, eager=eager_decode, many_steps=decode_many),
                eager_prefill=eager_prefill, parity=parity,
                e2e=dict(value=flops / (e2e_ms * 1e-3) / 1e12, unit=UNIT, ms_per_step=e2e_ms,
                         h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h, steps=e2e_steps,
                         overlap="copies in, compute and copies out of consecutive steps overlap (3 streams)"),
                gpu_launches=launches_per_step * args.steps,
                cpu_baseline=cpu)
    print(json.dumps(line))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_case(args):
    """A small single-kernel case for profiler captures: a few launches, nothing else."""
    import paper_2503_03588_b200 as pa

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    if args.case == "prefill32k":
        w = si.PREFILL_32K
        Q, K, V = (t.to(dev) for t in si.prefill_inputs(w))
        rp, ci = pa.pa_build_layout(w.seq_len, w.block, w.window_blocks, w.sink_blocks)
        o, lse, ws = pa.pa_prefill(Q, K, V, rp, ci)
        for _ in range(args.steps):
            pa.pa_prefill(Q, K, V, rp, ci, o=o, lse=lse, workspace=ws)
        pa.pa_prefill_status(ws)
    elif args.case == "backward32k":
        w = si.PREFILL_32K
        Q, K, V = (t.to(dev) for t in si.prefill_inputs(w))
        rp, ci = pa.pa_build_layout(w.seq_len, w.block, w.window_blocks, w.sink_blocks)
        o, lse, ws = pa.pa_prefill(Q, K, V, rp, ci)
        gen = torch.Generator(device=dev)
        gen.manual_seed(w.seed + 9)
        dO = torch.randn(o.shape, device=dev, dtype=torch.bfloat16, generator=gen)
        dq, dk, dv, wsb = pa.pa_prefill_backward(Q, K, V, o, lse, dO, rp, ci)
        for _ in range(args.steps):
            pa.pa_prefill_backward(Q, K, V, o, lse, dO, rp, ci, dq=dq, dk=dk, dv=dv, workspace=wsb)
        pa.pa_prefill_status(wsb)
    elif args.case == "decode_persist":
        # The persistent form of the decode row kernel on a case small enough for a full-set capture:
        # batch 96 (384 rows), 16K-token caches (1.6 GB), lengths uniform in [8192, 16384].
        wd = si.DECODE_B8
        batch, max_len = 96, 16384
        gen = torch.Generator(device=dev)
        gen.manual_seed(wd.seed + 96)
        kc = torch.randn((batch, max_len, wd.n_kv_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
        vc = torch.randn((batch, max_len, wd.n_kv_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
        qd = torch.randn((batch, wd.n_q_heads, wd.head_dim), device=dev, dtype=torch.bfloat16, generator=gen)
        lens = np.random.Generator(np.random.PCG64(wd.lens_seed + 96)).integers(max_len // 2, max_len + 1, size=batch)
        lens_d = torch.as_tensor(lens, dtype=torch.int32, device=dev)
        o, lse, ws = pa.pa_decode(qd, kc, vc, lens_d, wd.window_blocks, wd.sink_blocks)
        for _ in range(args.steps):
            pa.pa_decode(qd, kc, vc, lens_d, wd.window_blocks, wd.sink_blocks, o=o, lse=lse, workspace=ws)
        pa.pa_decode_status(ws)
    else:
        wd = si.DECODE_B8
        qd, kc, vc, lens = si.decode_inputs(wd)
        qd, kc, vc = qd.to(dev), kc.to(dev), vc.to(dev)
        lens_d = torch.as_tensor(lens, dtype=torch.int32, device=dev)
        o, lse, ws = pa.pa_decode(qd, kc, vc, lens_d, wd.window_blocks, wd.sink_blocks)
        for _ in range(args.steps):
            pa.pa_decode(qd, kc, vc, lens_d, wd.window_blocks, wd.sink_blocks, o=o, lse=lse, workspace=ws)
    torch.cuda.synchronize()
    print(json.dumps(dict(case=args.case, launches=args.steps + 1)))


def causal_csr(nqb: int):
    """Dense causal block layout: row i lists blocks 0..i."""
    lens = np.arange(1, nqb + 1, dtype=np.int64)
    row_ptr = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    col_idx = np.concatenate([np.arange(n, dtype=np.int32) for n in lens])
    return row_ptr, col_idx


def row_matched_window_csr(row_ptr_pa: np.ndarray):
    """Sliding window with the same number of blocks per row as the given layout: block 0 (sink)
    plus the most recent blocks, so both layouts have identical active-block counts."""
    nqb = len(row_ptr_pa) - 1
    cols = []
    for i in range(nqb):
        cnt = int(row_ptr_pa[i + 1] - row_ptr_pa[i])
        recent = np.arange(i - (cnt - 1) + 1, i + 1, dtype=np.int32) if cnt > 1 else np.zeros(0, np.int32)
        row = np.concatenate([[0], recent]).astype(np.int32) if cnt > 1 else np.array([i], np.int32)
        row = np.unique(np.clip(row, 0, i))
        while len(row) < cnt:  # early rows where the sink falls inside the window
            row = np.unique(np.concatenate([row, [max(0, int(row[1] if len(row) > 1 else row[0]) - 1)]])).astype(np.int32)
            if len(row) == i + 1:
                break
        cols.append(row.astype(np.int32))
    rp = np.concatenate([[0], np.cumsum([len(c) for c in cols])]).astype(np.int32)
    return rp, np.concatenate(cols)


def run_sweep(args):
    """Sequence-length sweep of the prefill kernel: the PowerAttention layout, dense causal and a
    row-matched sliding window (same active-block count) through the same pa_prefill call.
    Prints one JSON object per (length, layout)."""
    import paper_2503_03588_b200 as pa

    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = read_peaks()
    for N in si.SWEEP_SEQ_LENS:
        if N > args.sweep_max_len:
            continue
        w = si.sweep_workload(N)
        Q, K, V = (t.to(dev) for t in si.prefill_inputs(w))
        rp_pa, ci_pa = pa.pa_build_layout(N, w.block, w.window_blocks, w.sink_blocks)
        rp_host = rp_pa.cpu().numpy()
        nqb = len(rp_host) - 1
        layouts = {"powerattention": (rp_pa, ci_pa)}
        rw, cw = row_matched_window_csr(rp_host)
        layouts["sliding_window_row_matched"] = (torch.as_tensor(rw).to(dev), torch.as_tensor(cw).to(dev))
        # The paper's own block size (256 tokens, Section 4.1), listed by the kernel's 64-token tiles.
        layouts["powerattention_block256"] = pa.pa_build_tile_layout(N, 256, w.window_blocks, w.sink_blocks, w.block)
        if N <= args.sweep_dense_max_len:
            rc, cc = causal_csr(nqb)
            layouts["dense_causal"] = (torch.as_tensor(rc).to(dev), torch.as_tensor(cc).to(dev))
        o = lse = ws = None
        for name, (rp, ci) in layouts.items():
            nnz = int(ci.numel())
            o, lse, ws = pa.pa_prefill(Q, K, V, rp, ci, o=o, lse=lse, workspace=ws)
            reps = 3 if name == "dense_causal" else 10
            for _ in range(2):
                pa.pa_prefill(Q, K, V, rp, ci, o=o, lse=lse, workspace=ws)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(reps):
                pa.pa_prefill(Q, K, V, rp, ci, o=o, lse=lse, workspace=ws)
            e1.record()
            torch.cuda.synchronize()
            pa.pa_prefill_status(ws)
            ms = e0.elapsed_time(e1) / reps
            tf = block_pair_flops(nnz, w) / (ms * 1e-3) / 1e12
            print(json.dumps(dict(sweep=True, seq_len=N, layout=name, active_block_pairs=nnz, ms=ms, tflops=tf,
                                  frac_of_bf16_peak=tf / peaks["bf16_tflops"], peak_source=peaks["source"])), flush=True)
        del Q, K, V, o, lse


def spawn_replicas(n: int) -> int:
    """`python bench.py --gpus N` outside torchrun: start N replica processes of this script, one
    per GPU, with the rendezvous variables torchrun would set; rank 0's output is the job's line."""
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for rank in range(n):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable] + sys.argv, env=env))
    rc = 0
    for pr in procs:
        rc = rc or pr.wait()
    return rc


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--shard-heads", action="store_true",
                    help="with N > 1: split the one problem by KV heads over the ranks (strong scaling) instead of replicas")
    ap.add_argument("--no-decode-scale-up", action="store_true", help="skip the batch-64/256 decode lines")
    ap.add_argument("--case", default=None, choices=["prefill32k", "backward32k", "decode", "decode_persist"],
                    help="run only a small single-kernel case (for profiler captures)")
    ap.add_argument("--sweep", action="store_true", help="sequence-length sweep with comparison layouts")
    ap.add_argument("--sweep-max-len", type=int, default=262144)
    ap.add_argument("--sweep-dense-max-len", type=int, default=131072)
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.case:
        run_case(args)
        return
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_replicas(args.gpus))
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
