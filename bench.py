#!/usr/bin/env python
"""Benchmark of the Ecco decompression hot path on B200.

One step = one pass of the whole hot path over the Llama-2-7B-shaped configuration:
  1. ecco_decompress of the 7 compressed projection matrices of one decoder layer (one batched call),
  2. ecco_gemv (fused decode + GEMV) over the same 7 matrices at batch 1,
  3. the same at batch 8,
  4. ecco_attn_scores over the layer's compressed K cache [8][32][4096][128], one query per sequence,
  5. ecco_attn_values (softmax . V) over the layer's compressed V cache.
The headline `value` is the fp16 output rate of segment 1 (decompress output GB/s); the other
segments are reported beside it (GEMV microseconds per layer, attention microseconds).  After the
headline step a single-GPU run also times the long-context and the 70B-shaped configurations and
reports them under `other_configs`.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

N > 1: one process per GPU.  Started under torchrun the ranks are taken from its environment; started
directly, the script re-launches itself under torch.distributed.run with N processes on this node.
Every rank runs the same step on its own copy of the workload (the blocks of a tensor are independent,
so the path shards with no data-path collective: weak scaling); the time is the maximum over ranks of
the device time, the value the sum of the ranks' bytes over that time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

G, BLOCK = 128, 64
METRIC, UNIT = "decompress_output_GBps", "GB/s"


def parse_args(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--small", action="store_true", help="reduced workload for profiler captures (q and gate only, K cache batch 2; with --workload cfg5: batch-2 long-context caches)")
    ap.add_argument("--workload", default="cfg2", choices=["cfg2", "cfg4", "cfg5", "act2x", "var"],
                    help="cfg2 (default): Llama-2-7B-shaped layer + cfg3 K cache; cfg4: 70B-shaped MLP weights + stream-size "
                         "sweep; cfg5: long-context GQA K cache [16][8][32768][128] (decompress + attention scores with 8 "
                         "query heads per KV head); act2x: the 2x activation codec on a [32768][8192] fp16 tensor; var: the "
                         "variable-length container on the cfg2 gate/up/down matrices")
    ap.add_argument("--decompress-calls", choices=["batch", "single"], default="batch",
                    help="decompress segment: one ecco_decompress_batch call over the step's tensors (default) or one ecco_decompress per tensor")
    ap.add_argument("--gemv-calls", choices=["grouped", "single"], default="grouped",
                    help="GEMV segments: one ecco_gemv_batch call per group of matrices that a decoder layer can issue together "
                         "(q+k+v, o, gate+up, down; default) or one ecco_gemv call per matrix")
    ap.add_argument("--only", default="", help="comma list of segments to run: decompress,gemv1,gemv8,attn (profiling aid)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-configs", action="store_true", help="skip the cfg5 / cfg4 measurements that follow the headline step")
    return ap.parse_args(argv)


def relaunch_command(args, argv, environ):
    """--gpus N > 1 without a torchrun environment: the command that starts N ranks of this script on this node
    (None when no re-launch is needed).  A torchrun environment whose world size contradicts --gpus is an error."""
    world = environ.get("WORLD_SIZE")
    if world is not None:
        if args.gpus != int(world) and args.gpus != 1:
            raise SystemExit(f"--gpus {args.gpus} contradicts WORLD_SIZE={world}")
        return None
    if args.gpus <= 1:
        return None
    import socket

    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]


def cores() -> int:
    try:
        return max(1, len(os.sched_getaffinity(0)))
    except AttributeError:
        return os.cpu_count() or 1


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ------------------------------------------------------------------------------------------------
# clocks during the timed region
# ------------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "25", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()                  # the exact process started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0])); mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------
def oracle_sample_blocks(n_groups_wanted: int):
    """Oracle-only path: calibrate on the config-2 calibration matrix and encode the first rows of the
    q-projection-shaped matrix with the oracle's own encoder."""
    from oracle import ecco_oracle as eo
    from paper_2505_06901_b200 import synth

    cal = synth.weight_matrix(256, 1024, 2002)
    meta = eo.calibrate(cal, S=64, H=4, seed=2, select=eo.SELECT_MSE)
    rows = max(1, -(-n_groups_wanted // 32))
    w = synth.weight_matrix(rows, 4096, 1002 * 16)
    eo.set_exponent(meta, w)
    blocks, _ = eo.encode(meta, w.reshape(-1)[: n_groups_wanted * G], eo.SELECT_MSE)
    return eo, meta, blocks


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    c = cores()
    total = args.steps + args.warmup
    # about 60 s for the whole run at ~70k groups/s per core, at most 2^16 groups per step
    n = int(min(1 << 16, max(2048, 70000 * c * 60 // max(1, total))))
    n = min(n, 16384)                       # the oracle's own encoder prepares the sample (~1 s per 8k groups)
    eo, meta, blocks = oracle_sample_blocks(n)
    for _ in range(args.warmup):
        eo.decode_threads(meta, blocks, c)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        eo.decode_threads(meta, blocks, c)
    dt = time.perf_counter() - t0
    value = n * G * 2 * args.steps / dt / 1e9
    sample = f"{n} groups of a 4096-wide q-projection-shaped matrix (config-2 distribution), decoded {args.steps}x"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "cfg2 llama2-7b decoder layer + cfg3 K cache (bounded sample, CPU oracle)", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": c, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline(layer, c: int, kv_tensor=None):
    """The oracle's decoder on a bounded sample of the benchmark's own blocks (about 15 s of CPU work), and its
    decode + dot product for one GEMV sample and one attention-score sample."""
    from oracle import ecco_oracle as eo

    t = layer[0]
    S, e, pat, cb, kp = t.meta.tables()
    om = eo.Meta()
    om.S, om.H, om.e = S, 4, e
    for k in range(S):
        om.kp_len[k] = int(kp[k])
        for j in range(15):
            om.pattern[k][j] = int(pat.view(np.uint16)[k, j])
        for h in range(4):
            for s in range(16):
                om.cb_len[k][h][s] = int(cb[k, h, s])
    probe = t.blocks[:4096]
    t0 = time.perf_counter()
    eo.decode(om, probe)
    rate = 4096 / (time.perf_counter() - t0)          # groups/s on one core
    n = int(min(t.n_groups, max(8192, rate * 15)))
    t0 = time.perf_counter()
    eo.decode_threads(om, t.blocks[:n], c)
    dt = time.perf_counter() - t0
    out = {"value": n * G * 2 / dt / 1e9, "unit": UNIT, "cores": c, "kind": "oracle",
           "sample": f"first {n} groups of tensor '{t.name}' {tuple(t.shape)}, one pass on {c} threads",
           "groups_per_s": n / dt, "single_core_groups_per_s": rate}
    # the fused calls: the oracle's decode + fp64 dot products on one core, over the first rows of the same tensor
    # (and the first tokens of the K cache), a few seconds each
    from paper_2505_06901_b200 import synth

    fused = {}
    if len(t.shape) == 2:
        n_out, k = t.shape
        rows = int(max(32, min(n_out, rate * 3 // (k // G))))
        x = synth.activations(1, k, 11)
        t0 = time.perf_counter()
        eo.gemv(om, t.blocks[: rows * (k // G)], rows, k, x, 1)
        dt = time.perf_counter() - t0
        layer_weights = sum(int(np.prod(m.shape)) for m in layer if len(m.shape) == 2)
        fused["ecco_gemv batch 1"] = {"us_per_layer_equivalent": layer_weights * dt / (rows * k) * 1e6, "weights_per_s": rows * k / dt, "cores": 1,
                                      "sample": f"first {rows} rows of '{t.name}' {tuple(t.shape)}"}
    if kv_tensor is not None:
        kb, kh, kseq, _ = kv_tensor.shape
        S2, e2, pat2, cb2, kp2 = kv_tensor.meta.tables()
        km = eo.Meta()
        km.S, km.H, km.e = S2, 4, e2
        for k_ in range(S2):
            km.kp_len[k_] = int(kp2[k_])
            for j in range(15):
                km.pattern[k_][j] = int(pat2.view(np.uint16)[k_, j])
            for h in range(4):
                for s_ in range(16):
                    km.cb_len[k_][h][s_] = int(cb2[k_, h, s_])
        toks = int(max(256, min(kseq, rate * 3)))
        q = synth.queries(1, 1, 13)
        t0 = time.perf_counter()
        eo.attn_scores(km, kv_tensor.blocks[:toks], 1, 1, toks, 1, q, 128 ** -0.5)
        dt = time.perf_counter() - t0
        fused["ecco_attn_scores"] = {"tokens_per_s": toks / dt, "cores": 1, "sample": f"first {toks} tokens of head 0 of the K cache"}
    out["fused"] = fused
    return out


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
WORKLOADS = {
    "cfg2": dict(label="cfg2 llama2-7b decoder layer (q,k,v,o 4096x4096; gate,up 11008x4096; down 4096x11008; 1,581,056 groups) "
                       "+ cfg3 K and V caches [8][32][4096][128]",
                 step="decompress of the 7 matrices (one ecco_decompress_batch call), gemv batch 1 over the 7 matrices (four ecco_gemv_batch calls: q+k+v, o, gate+up, down), the same at batch 8, attn_scores x1 (K cache), attn_values x1 (V cache); --only kvcomp times ecco_kv_compress over the whole K cache",
                 l2="inputs larger than L2: each step streams 96.5 MiB of blocks and writes 386 MiB before any tensor is revisited"),
    "cfg4": dict(label="cfg4 llama-70b-shaped MLP weights (gate, up 28672x8192; down 8192x28672; 5,505,024 groups)",
                 step="decompress x3, gemv batch 1 x3; plus a decompress sweep over 64 MiB .. 4 GiB streams (stream_sweep)",
                 l2="inputs larger than L2: each step streams 336 MiB of blocks and writes 1.3 GiB"),
    "cfg5": dict(label="cfg5 long-context GQA K and V caches [16][8][32768][128] (4,194,304 groups each)",
                 step="decompress x1 (K), attn_scores x1 and attn_values x1 (8 query heads per KV head); --only kvcomp times ecco_kv_compress over the whole K cache",
                 l2="inputs larger than L2: each step streams 256 MiB of blocks and writes 1 GiB"),
    "small5": dict(label="reduced (profiling): cfg5-shaped K and V caches [2][8][16384][128], 8 query heads per KV head",
                   step="decompress x1 (K), attn_scores x1 and attn_values x1", l2="inputs larger than L2 for decompress only"),
    "small": dict(label="reduced (profiling): q + gate of cfg2, K cache [2][32][4096][128]",
                  step="decompress x2, gemv batch 1 x2, gemv batch 8 x2, attn_scores x1, attn_values x1",
                  l2="inputs larger than L2 except the q projection"),
}


def build_workload(name, workloads):
    """-> (weight tensors, kv tensor or None, q_per_kv, decompress_kv, default segments)."""
    if name == "cfg5":
        kt, vt = workloads.config5(which=("K", "V"), keep_source=True)
        vt.source = None
        return [], (kt, vt), 8, True, ["decompress", "attn", "attnv"]
    if name == "cfg4":
        return workloads.config4(), None, 1, False, ["decompress", "gemv1"]
    if name == "small5":
        base = workloads.calibrate_kv(5, 8)
        kt = workloads.kv_tensor("K", 2, 8, 16384, 1005 * 16, 3005, base, keep_source=True)
        vt = workloads.kv_tensor("V", 2, 8, 16384, 1005 * 16 + 1, 3005, base)
        return [], (kt, vt), 8, True, ["decompress", "attn", "attnv"]
    if name == "small":
        base = workloads.calibrate_kv(3, 32)
        kt = workloads.kv_tensor("K", 2, 32, 4096, 1003 * 16, 3003, base, keep_source=True)
        vt = workloads.kv_tensor("V", 2, 32, 4096, 1003 * 16 + 1, 3003, base)
        return workloads.config2(names=("q", "gate")), (kt, vt), 1, False, ["decompress", "gemv1", "gemv8", "attn", "attnv"]
    kt, vt = workloads.config3(which=("K", "V"), keep_source=True)
    vt.source = None
    return workloads.config2(), (kt, vt), 1, False, ["decompress", "gemv1", "gemv8", "attn", "attnv"]


def run_ours(args, workload=None, extras=True):
    """-> the JSON line of one workload as a dict (None on ranks other than 0).  extras = False skips the end-to-end
    leg, the per-tensor-call figure and the CPU baseline (used for the configurations after the headline step)."""
    import gc

    import torch

    from paper_2505_06901_b200 import binding as B
    from paper_2505_06901_b200 import distutil, synth, workloads

    rank, world, local = distutil.rank_info()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        if not dist.is_initialized():
            dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()

    # ---- workload (the same seeded tensors on every rank)
    workload = workload or args.workload
    wname = ("small5" if workload == "cfg5" else "small") if args.small else workload
    weights, kvt, q_per_kv, decompress_kv, default_segs = build_workload(wname, workloads)
    kt, vt = kvt if kvt is not None else (None, None)
    segs = [s for s in args.only.split(",") if s] or default_segs
    stream = torch.cuda.current_stream()
    need8 = "gemv8" in segs
    mats = []                                       # weight matrices: decompress + GEMV targets
    for t in weights:
        n_out, k = t.shape
        wsb = B.ecco_gemv_workspace_bytes(n_out, k, 8 if need8 else 1)
        mats.append(dict(t=t, n=t.n_groups, n_out=n_out, k=k, meta=B.meta_to_device(t.meta), blocks=torch.from_numpy(t.blocks).cuda(),
                         out=torch.empty(t.n_groups * G, dtype=torch.float16, device="cuda"),
                         x1=torch.from_numpy(synth.activations(1, k, 11)).cuda(), x8=torch.from_numpy(synth.activations(8, k, 12)).cuda(),
                         y1=torch.empty((1, n_out), dtype=torch.float32, device="cuda"),
                         y8=torch.empty((8, n_out), dtype=torch.float32, device="cuda"),
                         ws=torch.empty(wsb, dtype=torch.uint8, device="cuda"), wsb=wsb))
    dec = list(mats)                                # decompress targets
    kv = None
    if kt is not None:
        kb, kh, kseq, _ = kt.shape
        kv = dict(t=kt, n=kt.n_groups, meta=B.meta_to_device(kt.meta), blocks=torch.from_numpy(kt.blocks).cuda(),
                  q=torch.from_numpy(synth.queries(kb, kh * q_per_kv, 13)).cuda(),
                  scores=torch.empty((kb, kh * q_per_kv, kseq), dtype=torch.float32, device="cuda"))
        avb = B.ecco_attn_values_workspace_bytes(kb, kh, kseq, q_per_kv)
        kv.update(v_meta=B.meta_to_device(vt.meta), v_blocks=torch.from_numpy(vt.blocks).cuda(),
                  attn_out=torch.empty((kb, kh * q_per_kv, G), dtype=torch.float32, device="cuda"),
                  av_ws=torch.empty(avb, dtype=torch.uint8, device="cuda"), av_wsb=avb)
        if "kvcomp" in segs:
            kv.update(x=torch.from_numpy(kt.source.reshape(-1)).cuda(), cblocks=torch.empty((kt.n_groups, BLOCK), dtype=torch.uint8, device="cuda"))
        if decompress_kv:
            kv["out"] = torch.empty(kt.n_groups * G, dtype=torch.float16, device="cuda")
            dec.append(kv)

    dec_items = B.decompress_items([(d["meta"], d["blocks"], d["n"], d["out"]) for d in dec])      # marshalled once

    def seg_decompress_single():
        for d in dec:
            B.ecco_decompress(d["meta"], d["blocks"], d["n"], d["out"], stream)

    def seg_decompress():
        # the tensors of a layer are decompressed together: one ecco_decompress_batch call (one launch per 8 tensors)
        if args.decompress_calls == "batch":
            B.ecco_decompress_batch(dec_items, stream)
        else:
            seg_decompress_single()

    def seg_gemv_single(b):
        for d in mats:
            B.ecco_gemv(d["meta"], d["blocks"], d["n_out"], d["k"], d["x1" if b == 1 else "x8"], b, d["y1" if b == 1 else "y8"],
                        d["ws"], d["wsb"], stream)

    # The products of a decoder layer that do not depend on each other go out in one ecco_gemv_batch call: q, k and v
    # read the same activations, and so do gate and up; o and down each wait for what comes before them.
    by_name = {d["t"].name: d for d in mats}
    gemv_groups = [[by_name[n] for n in grp if n in by_name] for grp in (("q", "k", "v"), ("o",), ("gate", "up"), ("down",))]
    gemv_groups = [g for g in gemv_groups if g]
    if sum(len(g) for g in gemv_groups) != len(mats):
        gemv_groups = [[d] for d in mats]
    grouped = {}
    for b in (1, 8):
        if b == 8 and not need8:
            continue
        calls = []
        for g in gemv_groups:
            xk, yk = ("x1", "y1") if b == 1 else ("x8", "y8")
            items = [(d["meta"], d["blocks"], d["n_out"], d["k"], g[0][xk], d[yk]) for d in g]      # one x for the group
            nb = B.ecco_gemv_batch_workspace_bytes(items, b)
            calls.append((B.gemv_items(items), torch.empty(nb, dtype=torch.uint8, device="cuda"), nb))      # marshalled once
        grouped[b] = calls

    def seg_gemv(b):
        if args.gemv_calls == "grouped":
            for items, ws, nb in grouped[b]:
                B.ecco_gemv_batch(items, b, ws, nb, stream)
        else:
            seg_gemv_single(b)

    def seg_attn():
        if kv is not None:
            B.ecco_attn_scores(kv["meta"], kv["blocks"], kb, kh, kseq, q_per_kv, kv["q"], 128 ** -0.5, kv["scores"], stream)

    def seg_attnv():
        if kv is not None:
            B.ecco_attn_values(kv["v_meta"], kv["v_blocks"], kb, kh, kseq, q_per_kv, kv["scores"], kv["attn_out"], kv["av_ws"],
                               kv["av_wsb"], stream)

    def seg_kvcomp():
        if kv is not None:
            B.ecco_kv_compress(kv["meta"], kv["x"], kv["n"], kv["cblocks"], stream)

    def step(ev=None):
        if ev: ev[0].record(stream)
        if "decompress" in segs: seg_decompress()
        if ev: ev[1].record(stream)
        if "gemv1" in segs: seg_gemv(1)
        if ev: ev[2].record(stream)
        if "gemv8" in segs: seg_gemv(8)
        if ev: ev[3].record(stream)
        if "attn" in segs: seg_attn()
        if ev: ev[4].record(stream)
        if "attnv" in segs: seg_attnv()
        if ev: ev[5].record(stream)
        if "kvcomp" in segs: seg_kvcomp()
        if ev: ev[6].record(stream)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        step()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(7)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    launches0 = B.ecco_kernel_launch_count()
    barrier()
    for ev in events:
        step(ev)
    barrier()
    launches = B.ecco_kernel_launch_count() - launches0
    clocks = sampler.stop()
    assert B.ecco_device_status() == 0, "a kernel reported a device-side timeout"

    total_ms = events[0][0].elapsed_time(events[-1][6])
    seg_ms = [sum(ev[i].elapsed_time(ev[i + 1]) for ev in events) for i in range(6)]
    total_ms, dec_ms, g1_ms, g8_ms, at_ms, av_ms, kc_ms = distutil.max_over_ranks([total_ms] + seg_ms, dist, "cuda")   # slowest rank decides

    groups = sum(d["n"] for d in dec)
    out_bytes = groups * G * 2
    value = world * out_bytes * args.steps / (dec_ms / 1e3) / 1e9 if dec_ms > 0 else 0.0

    # ---- end to end through the C ABI with host buffers: H2D of the blocks, decompress, D2H of the fp16
    e2e = None
    if "decompress" in segs and dec and extras:
        h_in = [torch.from_numpy(d["t"].blocks).pin_memory() for d in dec]
        h_out = [torch.empty(d["n"] * G, dtype=torch.float16).pin_memory() for d in dec]

        # what a caller with host buffers does: three streams (copy in, decompress, copy out) chained by events per
        # tensor, so that the copies of one tensor run beside the kernel and the opposite copy of its neighbours
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in dec]
        ev_k = [torch.cuda.Event() for _ in dec]
        ev_out = [torch.cuda.Event() for _ in dec]
        for e in ev_k + ev_out:
            e.record(stream)

        def e2e_step():
            for i, (d, hi, ho) in enumerate(zip(dec, h_in, h_out)):
                s_in.wait_event(ev_k[i])                   # the previous decompress of these blocks has read them
                with torch.cuda.stream(s_in):
                    d["blocks"].copy_(hi, non_blocking=True)
                    ev_in[i].record(s_in)
                stream.wait_event(ev_in[i])
                stream.wait_event(ev_out[i])               # the previous copy-out of this output has finished
                B.ecco_decompress(d["meta"], d["blocks"], d["n"], d["out"], stream)
                ev_k[i].record(stream)
                s_out.wait_event(ev_k[i])
                with torch.cuda.stream(s_out):
                    ho.copy_(d["out"], non_blocking=True)
                    ev_out[i].record(s_out)

        def e2e_join():
            stream.wait_stream(s_in)
            stream.wait_stream(s_out)

        for _ in range(3):
            e2e_step()
        e2e_join()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        esteps = max(3, min(args.steps, 10))
        barrier()
        e0.record(stream)
        s_in.wait_event(e0)
        s_out.wait_event(e0)
        for _ in range(esteps):
            e2e_step()
        e2e_join()
        e1.record(stream)
        barrier()
        (ems,) = distutil.max_over_ranks([e0.elapsed_time(e1)], dist, "cuda")
        e2e = {"value": world * out_bytes * esteps / (ems / 1e3) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": groups * BLOCK, "d2h_bytes_per_step": out_bytes, "steps": esteps,
               "how": "pinned host buffers; H2D, ecco_decompress and D2H on three streams chained per tensor"}
        del h_in, h_out

    # ---- cfg4 only: standalone decompress over streams of 64 MiB .. 4 GiB (the gate matrix's blocks, tiled)
    sweep = None
    if wname == "cfg4" and rank == 0 and "decompress" in segs:
        gate = mats[0]
        sweep = []
        for mib in (64, 256, 1024, 4096):
            n = mib * (1 << 20) // BLOCK
            reps = -(-n // gate["n"])
            blocks = gate["blocks"].repeat(reps, 1)[:n].contiguous()
            out = torch.empty(n * G, dtype=torch.float16, device="cuda")
            for _ in range(2):
                B.ecco_decompress(gate["meta"], blocks, n, out, stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps_t = 5
            e0.record(stream)
            for _ in range(reps_t):
                B.ecco_decompress(gate["meta"], blocks, n, out, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            us = e0.elapsed_time(e1) * 1e3 / reps_t
            sweep.append({"compressed_MiB": mib, "groups": n, "us": us, "output_GBps": n * G * 2 / us / 1e3,
                          "hbm_frac": n * (BLOCK + G * 2) / us / 1e3 / measured_peaks()[0]})
            del blocks, out

    if rank != 0:
        if dist is not None and extras:
            dist.destroy_process_group()
        return None

    # the same tensors through one ecco_decompress call each, for the record
    single_us = None
    if "decompress" in segs and dec and args.decompress_calls == "batch" and extras:
        for _ in range(3):
            seg_decompress_single()
        s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        reps = max(3, min(args.steps, 20))
        barrier()
        s0.record(stream)
        for _ in range(reps):
            seg_decompress_single()
        s1.record(stream)
        barrier()
        (sms_,) = distutil.max_over_ranks([s0.elapsed_time(s1)], dist, "cuda")
        single_us = sms_ * 1e3 / reps

    # the GEMVs through one ecco_gemv call per matrix, for the record
    gemv_single_us = {}
    if args.gemv_calls == "grouped" and extras:
        for b, seg in ((1, "gemv1"), (8, "gemv8")):
            if seg not in segs or not mats:
                continue
            for _ in range(3):
                seg_gemv_single(b)
            s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(3, min(args.steps, 20))
            barrier()
            s0.record(stream)
            for _ in range(reps):
                seg_gemv_single(b)
            s1.record(stream)
            barrier()
            (gms_,) = distutil.max_over_ranks([s0.elapsed_time(s1)], dist, "cuda")
            gemv_single_us[f"batch{b}"] = gms_ * 1e3 / reps

    peak, peak_kind = measured_peaks()
    n_launch = max(1, -(-len(dec) // 8) if args.decompress_calls == "batch" else len(dec))
    avg_launch_s = dec_ms / 1e3 / (args.steps * n_launch) if dec_ms > 0 else float("nan")
    alg_bytes_per_launch = groups * (BLOCK + G * 2) / n_launch
    achieved = alg_bytes_per_launch / avg_launch_s / 1e9 if dec_ms > 0 else 0.0
    traffic = None
    ncu_consts = {}
    tp = os.path.join(ROOT, "paper_2505_06901_b200", "ncu_constants.json")
    if os.path.exists(tp):
        with open(tp) as f:
            ncu_consts = json.load(f)
        traffic = ncu_consts["decompress_dram"]["dram_bytes_per_group"] * groups / n_launch
    # What really limits the decoder are the SM's issue slots and its load/store pipe.  Their ceilings were measured
    # on this GPU with small probe kernels (warp instructions per clock per SM: 4.0 for adds and FFMA, 2.0 for the
    # logic / shift / permute / multiply-add instructions the decoder is made of; one shared-memory wavefront per
    # clock); the per-symbol costs are ncu counters of this kernel, the symbol rate is this run's.
    sm_limits = None
    if "decompress_sm" in ncu_consts and dec_ms > 0:
        # weights and KV caches cost differently per symbol (a KV cache has more code shapes, hence more escapes)
        c = ncu_consts.get("decompress_sm_weights", ncu_consts["decompress_sm"]) if wname in ("cfg2", "cfg4", "small") else ncu_consts["decompress_sm"]
        m = ncu_consts["measured_sm_rates"]
        props = torch.cuda.get_device_properties(local)
        sms, ghz = props.multi_processor_count, ((clocks or {}).get("sm_mhz") or 0) / 1e3
        if ghz > 0:
            warp_symbols_per_s = groups * (G / 32) * args.steps / (dec_ms / 1e3)
            sm_limits = {
                "issue": {"bound": "alu", "unit": "G warp-instr/s", "peak": sms * m["issue_warp_instr_per_clk_sm"] * ghz,
                          "achieved": warp_symbols_per_s * c["warp_instructions_per_warp_symbol"] / 1e9},
                "lsu": {"bound": "lsu", "unit": "G wavefronts/s", "peak": sms * m["lsu_wavefronts_per_clk_sm"] * ghz,
                        "achieved": warp_symbols_per_s * c["lsu_wavefronts_per_warp_symbol"] / 1e9},
                "per_warp_symbol": {"instructions": c["warp_instructions_per_warp_symbol"], "wavefronts": c["lsu_wavefronts_per_warp_symbol"],
                                    "captured_on": c["workload"]},
                "measured_rates": m,
                "source": "per-symbol costs: ncu capture of this kernel (paper_2505_06901_b200/ncu_constants.json); peaks = SMs x measured rate x sampled SM clock",
            }
            for k in ("issue", "lsu"):
                sm_limits[k]["frac"] = sm_limits[k]["achieved"] / sm_limits[k]["peak"]
    # the fused kernels against the same HBM peak (algorithmic bytes: blocks + vectors + results); what bounds them
    # is the SM load/store pipe, so the symbol rate is reported next to the HBM fraction
    seg_total = dec_ms + g1_ms + g8_ms + at_ms + av_ms + kc_ms
    kernels = []

    def kernel_entry(name, ms, alg_bytes_per_step, symbols_per_step):
        if ms <= 0 or symbols_per_step == 0:
            return
        sec = ms / 1e3 / args.steps
        kernels.append({"kernel": name, "share_of_step": ms / seg_total, "us_per_step": sec * 1e6,
                        "hbm_GBps": alg_bytes_per_step / sec / 1e9, "hbm_frac": alg_bytes_per_step / sec / 1e9 / peak,
                        "Gsymbols_per_s": symbols_per_step / sec / 1e9})

    w_groups = sum(d["n"] for d in mats)
    gemv_vec = lambda b: sum(2 * b * d["k"] + 4 * b * d["n_out"] for d in mats)
    kernel_entry("ecco_decompress", dec_ms if "decompress" in segs else 0, groups * (BLOCK + G * 2), groups * G)
    kernel_entry("ecco_gemv batch 1", g1_ms if "gemv1" in segs else 0, w_groups * BLOCK + gemv_vec(1), w_groups * G)
    kernel_entry("ecco_gemv batch 8", g8_ms if "gemv8" in segs else 0, w_groups * BLOCK + gemv_vec(8), w_groups * G)
    if kv is not None:
        kernel_entry(f"ecco_attn_scores q_per_kv {q_per_kv}", at_ms if "attn" in segs else 0, kv["n"] * (BLOCK + 4 * q_per_kv), kv["n"] * G)
        kernel_entry(f"ecco_attn_values q_per_kv {q_per_kv}", av_ms if "attnv" in segs else 0, kv["n"] * (BLOCK + 4 * q_per_kv), kv["n"] * G)
        kernel_entry("ecco_kv_compress", kc_ms if "kvcomp" in segs else 0, kv["n"] * (BLOCK + 2 * G), kv["n"] * G)
    info = WORKLOADS[wname]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": info["label"], "step": info["step"], "segments": segs, "l2": info["l2"],
                   "format": "S=64, H=4, group 128, 64-byte blocks"},
        "segments_us_per_step": {"decompress": dec_ms / args.steps * 1e3, "gemv_batch1": g1_ms / args.steps * 1e3,
                                 "gemv_batch8": g8_ms / args.steps * 1e3, "attn_scores": at_ms / args.steps * 1e3,
                                 "attn_values": av_ms / args.steps * 1e3, "kv_compress": kc_ms / args.steps * 1e3},
        "decompress_one_call_per_tensor_us": single_us,
        "gemv_us_per_layer_batch1": g1_ms / args.steps * 1e3 if wname == "cfg2" else None,
        "gemv_calls": ("ecco_gemv_batch per group: " + ", ".join("+".join(d["t"].name for d in g) for g in gemv_groups))
                      if args.gemv_calls == "grouped" else "one ecco_gemv per matrix",
        "gemv_one_call_per_matrix_us": gemv_single_us or None,
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": {"kernel": "ecco_decompress_tma_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                     "algorithmic_bytes_per_launch": alg_bytes_per_launch, "avg_launch_us": avg_launch_s * 1e6,
                     "note": "kernel of the headline metric; limited by the SM (issue slots and load/store pipe), not by HBM: see kernels[] and sm_limits"},
        "kernels": kernels,
    }
    if sm_limits is not None:
        line["sm_limits"] = sm_limits
    if "decompress" not in segs:
        # a diagnostic run without the headline segment has no headline number
        line["value"] = None
        line["roofline"] = None
        line["e2e"] = None
        line["note"] = "--only without decompress: the segment of the headline metric was not timed; see segments_us_per_step"
    if sweep is not None:
        line["stream_sweep"] = sweep
    if world == 1 and not args.no_cpu_baseline and dec and extras:
        line["cpu_baseline"] = cpu_baseline([d["t"] for d in dec], cores(), kt)
    if dist is not None and extras:
        dist.destroy_process_group()
    del mats, dec, kv, dec_items
    gc.collect()
    torch.cuda.empty_cache()
    return line


def other_config_summary(line):
    """What the default run keeps of a cfg4 / cfg5 measurement."""
    if line is None:
        return None
    keep = {"workload": line["config"]["workload"], "steps": line["steps"], "decompress_output_GBps": line["value"],
            "segments_us_per_step": {k: v for k, v in line["segments_us_per_step"].items() if v > 5.0},
            "kernels": line["kernels"], "clocks": line["clocks"],
            "roofline_frac": line["roofline"]["frac"] if line.get("roofline") else None}
    if "stream_sweep" in line:
        keep["stream_sweep"] = line["stream_sweep"]
    return keep


def run_var(args):
    """Variable-length container: one step = ecco_var_decompress of the cfg-2 gate, up and down matrices."""
    import torch

    from paper_2505_06901_b200 import binding as B
    from paper_2505_06901_b200 import distutil, workloads

    rank, world, local = distutil.rank_info()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    mats = []
    for t in workloads.config2(names=("gate", "up", "down"), keep_source=True):
        stream, index, total = B.ecco_var_encode_host(t.meta, t.source, B.SELECT_MSE | B.KEEP_EXPONENT)
        mats.append(dict(n=t.n_groups, meta=B.meta_to_device(t.meta), stream=torch.from_numpy(stream).cuda(), index=torch.from_numpy(index).cuda(),
                         blocks=torch.from_numpy(t.blocks).cuda(), out=torch.empty(t.n_groups * G, dtype=torch.float16, device="cuda"),
                         stream_bytes=stream.size, index_bytes=index.size, total_bits=total))
        t.source = None
    st = torch.cuda.current_stream()
    warmup = max(args.warmup, 3)

    def step(ev=None):
        if ev: ev[0].record(st)
        for d in mats:
            B.ecco_var_decompress(d["meta"], d["stream"], d["index"], d["n"], d["out"], st)
        if ev: ev[1].record(st)
        for d in mats:
            B.ecco_decompress(d["meta"], d["blocks"], d["n"], d["out"], st)
        if ev: ev[2].record(st)

    for _ in range(warmup):
        step()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    l0 = B.ecco_kernel_launch_count()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    for e in ev:
        step(e)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches = B.ecco_kernel_launch_count() - l0
    clocks = sampler.stop()
    v_ms = sum(e[0].elapsed_time(e[1]) for e in ev)
    b_ms = sum(e[1].elapsed_time(e[2]) for e in ev)
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    total_ms, v_ms, b_ms = distutil.max_over_ranks([total_ms, v_ms, b_ms], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peaks()
    groups = sum(d["n"] for d in mats)
    alg = sum(d["stream_bytes"] + 4 * d["n"] + d["n"] * G * 2 for d in mats)     # stream + 4-byte start per group + fp16 out
    v_s = v_ms / 1e3 / args.steps
    line = {
        "metric": "var_decompress_output_GBps", "value": world * groups * G * 2 / v_s / 1e9, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "variable-length container of the cfg2 gate, up (11008x4096) and down (4096x11008) matrices",
                   "step": "ecco_var_decompress x3, then ecco_decompress x3 of the same matrices as 64-byte blocks (for comparison)",
                   "l2": "inputs larger than L2: 63 MiB of stream and 258 MiB of output per segment",
                   "mean_bits_per_group": sum(d["total_bits"] for d in mats) / groups},
        "segments_us_per_step": {"var_decompress": v_ms / args.steps * 1e3, "block_decompress": b_ms / args.steps * 1e3},
        "clocks": clocks, "gpu_launches": int(launches), "e2e": None,
        "roofline": {"kernel": "ecco_var_decompress_kernel", "bound": "hbm", "achieved": alg / v_s / 1e9, "peak": peak, "unit": "GB/s",
                     "frac": alg / v_s / 1e9 / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                     "algorithmic_bytes_per_launch": alg / len(mats), "avg_launch_us": v_s * 1e6 / len(mats)},
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_act2x(args):
    """2x activation codec (Sec. 3.2): one step = compress + decompress of a [32768][8192] fp16 N(0,1) tensor."""
    import torch

    from paper_2505_06901_b200 import binding as B
    from paper_2505_06901_b200 import distutil, synth

    rank, world, local = distutil.rank_info()
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    rows, cols = 32768, 8192
    x = synth.activations(rows, cols, 1006)
    n = rows * cols // 64
    d_x = torch.from_numpy(x).cuda()
    d_blocks = torch.empty((n, 64), dtype=torch.uint8, device="cuda")
    d_out = torch.empty_like(d_x)
    stream = torch.cuda.current_stream()
    warmup = max(args.warmup, 3)
    for _ in range(warmup):
        B.ecco_act_compress(d_x, n, d_blocks, stream)
        B.ecco_act_decompress(d_blocks, n, d_out, stream)
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    l0 = B.ecco_kernel_launch_count()
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    for e in ev:
        e[0].record(stream)
        B.ecco_act_compress(d_x, n, d_blocks, stream)
        e[1].record(stream)
        B.ecco_act_decompress(d_blocks, n, d_out, stream)
        e[2].record(stream)
    if dist is not None:
        dist.barrier()
    torch.cuda.synchronize()
    launches = B.ecco_kernel_launch_count() - l0
    clocks = sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    c_ms = sum(e[0].elapsed_time(e[1]) for e in ev)
    d_ms = sum(e[1].elapsed_time(e[2]) for e in ev)
    total_ms, c_ms, d_ms = distutil.max_over_ranks([total_ms, c_ms, d_ms], dist, "cuda")
    # end to end: blocks from pinned host memory, fp16 back to pinned host memory
    h_in, h_out = torch.empty((n, 64), dtype=torch.uint8).pin_memory(), torch.empty((rows, cols), dtype=torch.float16).pin_memory()
    h_in.copy_(d_blocks)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    esteps = 5
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(esteps):
        d_blocks.copy_(h_in, non_blocking=True)
        B.ecco_act_decompress(d_blocks, n, d_out, stream)
        h_out.copy_(d_out, non_blocking=True)
    e1.record(stream)
    torch.cuda.synchronize()
    (ems,) = distutil.max_over_ranks([e0.elapsed_time(e1)], dist, "cuda")
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return
    peak, peak_kind = measured_peaks()
    out_bytes = n * 128
    dec_s = d_ms / 1e3 / args.steps
    achieved = n * 192 / dec_s / 1e9
    line = {
        "metric": "act2x_decompress_output_GBps", "value": world * out_bytes / dec_s / 1e9, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "2x activation codec, fp16 N(0,1) [32768][8192] (4,194,304 groups of 64)",
                   "step": "ecco_act_compress x1, ecco_act_decompress x1",
                   "l2": "inputs larger than L2: 512 MiB of fp16, 256 MiB of blocks"},
        "segments_us_per_step": {"act_compress": c_ms / args.steps * 1e3, "act_decompress": d_ms / args.steps * 1e3},
        "clocks": clocks, "gpu_launches": int(launches),
        "e2e": {"value": world * out_bytes * esteps / (ems / 1e3) / 1e9, "unit": UNIT, "h2d_bytes_per_step": n * 64,
                "d2h_bytes_per_step": out_bytes, "steps": esteps},
        "roofline": {"kernel": "ecco_act_decompress_kernel", "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": None,
                     "algorithmic_bytes_per_launch": n * 192, "avg_launch_us": dec_s * 1e6},
        "kernels": [{"kernel": "ecco_act_compress", "us_per_step": c_ms / args.steps * 1e3,
                     "hbm_GBps": n * 192 / (c_ms / 1e3 / args.steps) / 1e9, "hbm_frac": n * 192 / (c_ms / 1e3 / args.steps) / 1e9 / peak},
                    {"kernel": "ecco_act_decompress", "us_per_step": dec_s * 1e6, "hbm_GBps": achieved, "hbm_frac": achieved / peak}],
    }
    if world == 1 and not args.no_cpu_baseline:
        from oracle import ecco_oracle as eo

        blocks = d_blocks[: 1 << 20].cpu().numpy()
        t0 = time.perf_counter()
        eo.act_decode(blocks)
        dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": blocks.shape[0] * 128 / dt / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"first {blocks.shape[0]} groups, one pass on one thread"}
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    a = parse_args(argv)
    cmd = relaunch_command(a, argv, os.environ)
    if cmd is not None:                                    # --gpus N without torchrun: start the N ranks here
        env = dict(os.environ, NCCL_DEBUG=os.environ.get("NCCL_DEBUG", "WARN"))
        raise SystemExit(subprocess.call(cmd, env=env))
    if a.impl == "reference":
        run_reference(a)
    elif a.workload == "act2x":
        run_act2x(a)
    elif a.workload == "var":
        run_var(a)
    else:
        world = int(os.environ.get("WORLD_SIZE", "1"))
        others = a.workload == "cfg2" and not a.small and not a.only and not a.no_other_configs and world == 1
        line = run_ours(a)
        if line is not None and others:
            # the long-context and the 70B-shaped configurations, outside the headline step (fewer steps, no end-to-end leg)
            short = argparse.Namespace(**vars(a))
            short.steps, short.warmup = max(3, min(a.steps, 10)), 3
            line["other_configs"] = {w: other_config_summary(run_ours(short, workload=w, extras=False)) for w in ("cfg5", "cfg4")}
        if line is not None:
            print(json.dumps(line))


if __name__ == "__main__":
    main()
