#!/usr/bin/env python
"""Benchmark of the BlossomRec sparse-attention hot path (selection + forward + backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 4] [--impl ours|reference]

One "step" = one pass of the whole hot path over one synthetic batch: block summary + scoring
+ top-k selection, the fused two-branch forward (training mode: per-branch outputs and
log-sum-exps saved) and the backward.  Prints ONE JSON line (rank 0).

value     tokens/s with every input already resident in HBM (CUDA events, max over ranks)
e2e       the same metric with HOST (pinned) inputs: host->device copies of q, k, v, dout, gate
          and device->host copies of out, dq, dk, dv, dgate inside the timed region
roofline  the kernel with the largest share of the timed region: its algorithmic FLOPs (or
          bytes) per launch over its average device time (per-launch CUDA events recorded by
          the library inside the timed region) against the measured peak of this machine
cpu_baseline  the fp64 oracle, as it stands, on the host cores, on a bounded sample
N > 1     every rank runs the same batch on its own GPU (independent replicas, no collective
          on the data path): weak scaling, value = N * tokens / max-over-ranks time.
--impl reference  times the oracle itself (rank 0 only), same metric and config.
"""
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

METRIC = "sparse-attn fwd+bwd tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------ algorithmic work model
def work_model(w):
    """Visited (query block, key block) tiles and the FLOPs / bytes they imply.

    tile FLOPs = 2 * Bk * Bk * D per GEMM per visited tile and branch; forward 2 GEMMs
    (QK^T, PV), backward 5 (S recompute, dP, dV, dK, dQ).  Compulsory bytes: forward reads
    q, k, v and writes out, out_lt, out_st (+ lse, indices); backward reads q, k, v, dout,
    out_lt, out_st, lse and writes dq, dk, dv: 15 q-shaped tensors in total (with grouped
    key/value heads the k-, v-, dk- and dv-shaped ones are kv_heads / heads as large).
    """
    import numpy as np
    M, Bk = w.n_blocks, w.block
    lens = np.full(w.B, w.L) if w.seq_lens is None else w.seq_lens.astype(np.int64)
    tiles_L = tiles_S = 0
    for ln in np.unique(lens):
        cnt = int((lens == ln).sum())
        pad0 = w.L - int(ln)
        first = pad0 // Bk if ln > 0 else M
        tl = ts = 0
        for qb in range(first, M):
            tl += min(w.topk, qb - first + 1)
            lo_pos = max(pad0, qb * Bk - (w.window - 1))
            ts += qb - lo_pos // Bk + 1
        if w.stis_mode == 1:
            # power-law mask: the work is counted per (query, key) pair of Eq. 15 and expressed in
            # tiles of Bk x Bk pairs (fractional), since its links do not fill tiles
            t = np.arange(pad0, w.L)
            pairs = np.minimum(t - pad0 + 1, w.window).astype(np.float64)
            blk, r = w.stis_block, 0
            while (1 << r) * blk <= w.L:
                d = 1 << r
                kb = t // blk - d                      # the key block at distance 2^r
                lo = np.maximum(kb * blk, pad0)
                hi = np.minimum(kb * blk + blk - 1, t - w.window)   # keys the window does not hold already
                pairs += np.maximum(hi - lo + 1, 0) * (kb >= 0)
                r += 1
            lastlo = np.maximum(w.L - blk, pad0)
            own = (t // blk) * blk                       # last-block keys: distance 0 only, beyond the window
            pairs += np.maximum(np.minimum(t - w.window, t) - np.maximum(lastlo, own) + 1, 0) * (t >= lastlo)
            ts = float(pairs.sum()) / (Bk * Bk)
        tiles_L += cnt * tl * w.H
        tiles_S += cnt * ts * w.H
    esz = 2 if w.dtype == "bf16" else 4
    T = w.B * w.H * w.L * w.D * esz
    Tk = T * (w.kv_heads or w.H) // w.H          # a k- or v-shaped tensor
    tile_flops = 2.0 * Bk * Bk * w.D
    tb = tiles_L + tiles_S
    lse_b = 2 * w.B * w.H * w.L * 4
    idx_b = w.B * (w.kv_heads or w.H) * M * w.topk * 4
    gemms = {"fwd": 2, "bwd": 5, "fwd_simt": 2, "fwd_tc": 2, "bwd_dq_simt": 3, "bwd_dkdv_simt": 2,
             "bwd_dq_tc": 3, "bwd_dkdv_tc": 2}
    byts = {"fwd": 4 * T + 2 * Tk + lse_b + idx_b, "bwd": 5 * T + 4 * Tk + 2 * lse_b + idx_b}
    byts.update({"fwd_simt": byts["fwd"], "fwd_tc": byts["fwd"],
                 "bwd_dq_simt": 5 * T + 2 * Tk + 2 * lse_b, "bwd_dkdv_simt": 2 * T + 4 * Tk + 2 * lse_b,
                 "bwd_dq_tc": 5 * T + 2 * Tk + 2 * lse_b, "bwd_dkdv_tc": 2 * T + 4 * Tk + 2 * lse_b,
                 "summary": Tk, "score_select": T, "score_fast": T, "bwd_prep": 3 * T + lse_b,
                 "tc_meta": idx_b})
    return {"tiles_lt": tiles_L, "tiles_st": tiles_S, "tile_flops": tile_flops,
            "flops": {k: g * tb * tile_flops for k, g in gemms.items()}, "bytes": byts,
            "step_flops": 7 * tb * tile_flops, "step_bytes": 9 * T + 6 * Tk + 3 * lse_b + 2 * idx_b}


# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the attention kernels come
# from an ncu capture whose summary sits under profiles/ (the file gives the command and the date).
# It was taken at batch 4 of the long-history case (255 MB of tensors, more than L2); traffic grows
# in proportion to the batch, so a launch at batch B is charged B / 4 times these figures.  The
# file also records a hash of the kernel sources at capture time: once a kernel has changed the
# figure is stale and `traffic` is reported as null.  Other workloads and kernels report null.
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "cfg4_b4_dram_traffic.txt")
KERNEL_SOURCES = ("attn_tc_fwd.cu", "attn_tc_bwd.cu", "attn_tc_meta.cu", "tc_common.cuh", "tc_host.cu")


def kernel_source_hash():
    import hashlib
    h = hashlib.sha256()
    for name in KERNEL_SOURCES:
        with open(os.path.join(ROOT, "paper_2512_13368_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def load_traffic():
    """{kernel: bytes per launch at batch 4}, the capture's date; ({}, None) if absent or stale."""
    try:
        kv = dict(line.split(None, 1) for line in open(TRAFFIC_FILE) if line.strip() and line[0] != "#")
    except OSError:
        return {}, None
    if kv.get("source_hash", "").strip() != kernel_source_hash():
        return {}, None
    out = {k: float(v) for k, v in kv.items() if k in ("fwd_tc", "bwd_dq_tc", "bwd_dkdv_tc")}
    return out, kv.get("captured", "").strip() or None


# ------------------------------------------------------------------------ clock sampling
class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1]))
                    mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, val in zip(names, f[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons),
                       samples=len(sm))
        return out


# ------------------------------------------------------------------------- oracle timing
def oracle_sample(w, max_batch):
    """The bounded sample of the workload the oracle is timed on: its first `max_batch`
    batch entries (all heads)."""
    from paper_2512_13368_b200.workloads import Workload
    nb = min(max_batch, w.B)
    sl = None if w.seq_lens is None else w.seq_lens[:nb].copy()
    return Workload(w.name + f"[first {nb} of {w.B} batch entries]", w.dtype, nb, w.H, w.L, w.D,
                    w.block, w.topk, w.window, w.seed, w.q[:nb], w.k[:nb], w.v[:nb], w.gate,
                    w.dout[:nb], sl, w.stis_mode, w.stis_block, w.cmp_block, w.cmp_stride, w.kv_heads)


def time_oracle(ws):
    import oracle
    t0 = time.perf_counter()
    idx = None
    grouped = bool(ws.kv_heads) and ws.kv_heads != ws.H
    if (ws.cmp_block or ws.cmp_stride) and not grouped:   # selection through overlapping compression blocks (Eq. 8-11)
        idx = oracle.select_blocks_cmp(ws.q, ws.k, ws.block, ws.topk, ws.cmp_block or ws.block,
                                       ws.cmp_stride or ws.block, ws.seq_lens)
    if grouped:   # grouped key/value heads: one selection per group (Eq. 12)
        f = oracle.forward_gqa(ws.q, ws.k, ws.v, ws.gate, ws.block, ws.topk, ws.window, ws.seq_lens,
                               cmp_block=ws.cmp_block, cmp_stride=ws.cmp_stride,
                               stis_mode=ws.stis_mode, stis_block=ws.stis_block)
        oracle.backward_gqa(ws.q, ws.k, ws.v, ws.gate, ws.block, ws.topk, ws.window, f, ws.dout,
                            ws.seq_lens, stis_mode=ws.stis_mode, stis_block=ws.stis_block)
        return time.perf_counter() - t0
    oracle.forward_backward(ws.q, ws.k, ws.v, ws.gate, ws.dout, ws.block, ws.topk, ws.window,
                            ws.seq_lens, idx=idx, stis_mode=ws.stis_mode, stis_block=ws.stis_block)
    return time.perf_counter() - t0


SAMPLE_BATCH = {1: 4, 2: 256, 3: 128, 4: 16, 5: 128}  # batch entries the oracle is timed on (a few to ~10 s of host work)


def run_reference(args, w, cfg_desc):
    import oracle
    ws = oracle_sample(w, SAMPLE_BATCH[args.config])
    for _ in range(args.warmup):
        time_oracle(ws)
    times = [time_oracle(ws) for _ in range(args.steps)]
    sec = sum(times) / len(times)
    value = ws.tokens / sec
    cores = min(oracle.threads(), ws.B * ws.H)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": cfg_desc,
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle",
                             "sample": ws.name},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


# ------------------------------------------------------------------ replicas on several GPUs
def rank_max(x, world, device):
    """The slowest rank's value of x (a time): every rank returns the same number."""
    if world > 1:
        import torch
        import torch.distributed as dist
        t = torch.tensor([x], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return x


def replicas_tokens_per_s(world, tokens_per_replica, ms_per_step):
    """Whole-job throughput of `world` independent replicas that all take the slowest rank's
    time per step (weak scaling: the work per GPU is fixed)."""
    return world * tokens_per_replica / (ms_per_step * 1e-3)


# --------------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=4, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--short-term", default="window", choices=["window", "power-law"],
                    help="short-term branch: the configuration's causal window (headline) or the "
                         "power-law mask of Eq. 15 with --mask-window and --mask-block")
    ap.add_argument("--mask-window", type=int, default=8, help="w of the power-law mask (paper: 8 blocks of 1)")
    ap.add_argument("--mask-block", type=int, default=1, help="blk of the power-law mask")
    ap.add_argument("--cmp-block", type=int, default=0,
                    help="length l of overlapping compression blocks for the selection (Eq. 8, 11); 0 = off")
    ap.add_argument("--cmp-stride", type=int, default=0, help="their stride s")
    ap.add_argument("--kv-heads", type=int, default=0,
                    help="key/value heads shared by groups of query heads (0: one per query head)")
    ap.add_argument("--paper-options", action="store_true",
                    help="the paper's options together on the chosen shape: heads on 2 key/value heads, "
                         "compression blocks of 2 x block at stride block / 2, power-law mask (window 8, block 1)")
    ap.add_argument("--per-query", action="store_true",
                    help="one selection per query position (Eq. 13 as printed)")
    ap.add_argument("--learned-summary", action="store_true",
                    help="softmax-pooled block summaries (Eq. 9) with seeded pooling logits")
    ap.add_argument("--input-gate", action="store_true",
                    help="input-dependent gate (Eq. 18, one linear layer)")
    ap.add_argument("--non-causal", action="store_true",
                    help="no causal mask (bidirectional encoder)")
    ap.add_argument("--rope-theta", type=float, default=0.0,
                    help="rotate q and k by position inside the library (0 = off)")
    ap.add_argument("--no-secondary", action="store_true",
                    help="skip the L = 1024 case that the default run times beside the headline")
    ap.add_argument("--batch", type=int, default=0,
                    help="override the batch size (profiling captures on a smaller case; not a bench line)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    from paper_2512_13368_b200 import workloads
    if args.impl == "reference" and rank != 0:
        return 0
    kw = {}
    if args.batch and args.config != 1:
        kw["B"] = args.batch
    if args.kv_heads and args.config != 1:
        kw["kv_heads"] = args.kv_heads
    if args.paper_options and args.config != 1:
        kw["kv_heads"] = args.kv_heads or 2
        args.short_term = "power-law"
    w = workloads.CONFIGS[args.config](**kw)
    if args.paper_options and args.config != 1:
        args.cmp_block, args.cmp_stride = args.cmp_block or 2 * w.block, args.cmp_stride or w.block // 2
    if w.kv_heads:
        w.name += f"+kv_heads{w.kv_heads}"
    if args.short_term == "power-law":
        w.stis_mode, w.stis_block, w.window = 1, args.mask_block, args.mask_window
        w.name += f"+powerlaw(w{args.mask_window},blk{args.mask_block})"
    if args.cmp_block or args.cmp_stride:
        w.cmp_block, w.cmp_stride = args.cmp_block or w.block, args.cmp_stride or w.block
        w.name += f"+cmp(l{w.cmp_block},s{w.cmp_stride})"
    import numpy as np
    opt_rng = np.random.default_rng(1000 + w.seed)   # inputs of the options below, seeded like the rest
    if args.per_query:
        w.per_query = 1
        w.name += "+per-query-selection"
    if args.learned_summary:
        w.phi_logits = opt_rng.standard_normal(w.cmp_block or w.block).astype(np.float32)
        w.name += "+softmax-pooled-summary"
    if args.input_gate:
        w.gate_mode = 1
        w.gate = (opt_rng.standard_normal((w.H, 2 * w.D + 1)) / np.sqrt(w.D)).astype(np.float32)
        w.name += "+input-gate"
    if args.non_causal:
        w.causal = 0
        w.name += "+non-causal"
    if args.rope_theta > 0:
        w.rope_theta = float(args.rope_theta)
        w.name += f"+rope({args.rope_theta:g})"
    cfg_desc = {"workload": w.name, "batch": w.B, "heads": w.H, "kv_heads": w.kv_heads or w.H, "seq_len": w.L, "head_dim": w.D,
                "block_size": w.block, "top_k": w.topk, "window": w.window, "short_term": args.short_term,
                "mask_block": w.stis_block if w.stis_mode else None,
                "cmp_block": w.cmp_block or None, "cmp_stride": w.cmp_stride or None, "storage": w.dtype,
                "padding": "left, lengths U{5..200}" if w.seq_lens is not None else "none",
                "l2": "no flush: a step touches ~1 GB of distinct tensors, more than the 126 MB L2"
                if w.B * w.H * w.L * w.D * 2 * 15 > 4 * 126e6 else
                "working set fits L2; a 256 MB buffer is written between timed steps"}
    if args.impl == "reference":
        if args.steps == 20 and args.warmup == 5:
            args.steps, args.warmup = 3, 1
        run_reference(args, w, cfg_desc)
        return 0

    import torch
    from paper_2512_13368_b200 import binding, runner
    binding.load()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU fallback)"
    args.warmup = max(args.warmup, 3)
    dev = torch.device("cuda", local_rank if world > 1 else 0)
    torch.cuda.set_device(dev)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x):
        return rank_max(x, world, dev)

    peaks, peak_kind = load_peaks()

    def timed_run(w, steps, warmup):
        """K timed steps of one workload with device-resident inputs; returns the problem, the time
        per step (max over ranks), the launch count, the clock record and the roofline object."""
        p = runner.DeviceProblem(w, device=dev)
        model = work_model(w)
        flush = None
        if w.B * w.H * w.L * w.D * 2 * 15 <= 4 * 126e6:   # working set within reach of L2: flush it
            flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

        def step():
            if flush is not None:
                flush.fill_(1)
            p.step()

        for _ in range(warmup):
            step()
        barrier()
        # per-launch events recorded by the library inside the timed region
        sampler = ClockSampler(dev.index)
        sampler.start()
        time.sleep(0.3)
        launches0 = binding.blossom_launch_count()
        cap = 32 * steps
        # An event record between two kernels costs a few microseconds and keeps the second from
        # becoming resident before the first has ended, so only every 4th launch of each kernel
        # (= every 4th step) is bracketed: the other steps run as a user's would.
        every = 4 if steps >= 8 else 1
        binding.blossom_profile_every(every)
        binding.blossom_profile_start(cap)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        step_events = []
        barrier()
        e0.record()
        for _ in range(steps):
            if flush is not None:
                ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                flush.fill_(1)
                ea.record()
                p.step()
                eb.record()
                step_events.append((ea, eb))
            else:
                p.step()
        e1.record()
        barrier()
        launches = binding.blossom_launch_count() - launches0
        per_launch = binding.blossom_profile_stop(cap)
        binding.blossom_profile_every(1)
        if step_events:
            total_ms = sum(x.elapsed_time(y) for x, y in step_events)
        else:
            total_ms = e0.elapsed_time(e1)
        clocks = sampler.stop()
        assert binding.blossom_device_status(p.workspace) == 0
        ms_per_step = max_over_ranks(total_ms / steps)

        # ---- roofline of the kernel with the largest share
        agg = {}
        for name, ms in per_launch:
            e = agg.setdefault(name, [0, 0.0])
            e[0] += 1
            e[1] += ms
        tot_kernel_ms = sum(v[1] for v in agg.values()) or 1.0
        top = max(agg, key=lambda k: agg[k][1])
        avg_ms = agg[top][1] / agg[top][0]
        fl, by = model["flops"].get(top, 0.0), model["bytes"].get(top, 0.0)
        # A kernel timed per launch at full clocks with no power cap active is held against the
        # burst matmul peak (taken under the same conditions); a capped run against the sustained one.
        capped = "sw_power_cap" in clocks["reasons"] or (
            clocks["sm_mhz"] is not None and clocks["sm_mhz"] < 0.95 * (clocks["sm_max_mhz"] or 1))
        tensor_peak = peaks["bf16_tflops_sustained"] if capped else peaks["bf16_tflops"]
        hbm_peak = peaks["hbm_gbs"]
        if fl / (tensor_peak * 1e12) >= by / (hbm_peak * 1e9):
            ach = fl / (avg_ms * 1e-3) / 1e12
            roof = {"bound": "tensor", "achieved": ach, "peak": tensor_peak, "unit": "TFLOP/s",
                    "frac": ach / tensor_peak}
        else:
            ach = by / (avg_ms * 1e-3) / 1e9
            roof = {"bound": "hbm", "achieved": ach, "peak": hbm_peak, "unit": "GB/s", "frac": ach / hbm_peak}
        plain_cfg4 = w.name == "cfg4-long"
        table, captured = load_traffic() if plain_cfg4 else ({}, None)
        traffic = table.get(top)
        roof.update({"traffic": traffic * w.B / 4 if traffic else None, "traffic_captured": captured if traffic else None,
                     "kernel": top, "kernel_ms": avg_ms, "kernel_share": agg[top][1] / tot_kernel_ms,
                     "events": ("every 4th launch of each kernel in the timed region bracketed by events (one step in four)"
                                if every == 4 else "every launch in the timed region bracketed by events"),
                     "peak_source": (f"of {peak_kind}: " + ("sustained bf16 matmul (power cap or reduced clocks seen)"
                                                           if capped else "burst bf16 matmul (full clocks, no cap)")
                                     + " / copy bandwidth"),
                     "kernels": {k: {"launches": v[0], "ms_per_launch": v[1] / v[0],
                                     "share": v[1] / tot_kernel_ms} for k, v in sorted(agg.items())}})
        non_gemm = sum(v[1] * every / steps for k, v in agg.items()
                       if k in ("summary", "score_select", "score_fast", "tc_meta", "bwd_prep", "gate_grad"))
        t_roof = max(model["step_flops"] / (tensor_peak * 1e12), model["step_bytes"] / (hbm_peak * 1e9))
        t_sus = max(model["step_flops"] / (peaks["bf16_tflops_sustained"] * 1e12), model["step_bytes"] / (hbm_peak * 1e9))
        roof["step"] = {"roofline_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms_per_step,
                        "frac_vs_sustained_peak": t_sus * 1e3 / ms_per_step,
                        "bound": "tensor" if model["step_flops"] / (tensor_peak * 1e12) >= model["step_bytes"] / (hbm_peak * 1e9) else "hbm",
                        "tile_gflop": model["step_flops"] / 1e9, "hbm_mb": model["step_bytes"] / 1e6,
                        "non_gemm_kernels_ms": non_gemm}
        return p, step, ms_per_step, launches, clocks, roof

    p, step, ms_per_step, launches, clocks, roof = timed_run(w, args.steps, args.warmup)
    value = replicas_tokens_per_s(world, w.tokens, ms_per_step)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    # ---- the same K steps replayed from one captured CUDA graph (no per-launch events, no host
    # work between kernels); reported beside the headline, which stays the eager, event-timed run
    graph_info = None
    try:
        side = torch.cuda.Stream(dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            p.step()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=side):
                step()
        torch.cuda.current_stream().wait_stream(side)
        for _ in range(3):
            g.replay()
        barrier()
        e0.record()
        for _ in range(args.steps):
            g.replay()
        e1.record()
        barrier()
        g_ms = max_over_ranks(e0.elapsed_time(e1) / args.steps)
        graph_info = {"ms_per_step": g_ms, "value": replicas_tokens_per_s(world, w.tokens, g_ms), "unit": "tokens/s"}
        del g
    except Exception as exc:  # the headline does not depend on it
        graph_info = {"error": str(exc)[:200]}

    # ---- the other sequence length the metric names (L = 1024, the mid-length case), timed the
    # same way in the same process and reported beside the headline
    secondary = None
    if args.config == 4 and not args.no_secondary and w.name == "cfg4-long":
        del p
        torch.cuda.empty_cache()
        w3 = workloads.config3()
        _p3, _s3, ms3, l3, clk3, roof3 = timed_run(w3, args.steps, args.warmup)
        secondary = {"workload": w3.name, "batch": w3.B, "heads": w3.H, "seq_len": w3.L, "head_dim": w3.D,
                     "block_size": w3.block, "top_k": w3.topk, "window": w3.window,
                     "ms_per_step": ms3, "value": replicas_tokens_per_s(world, w3.tokens, ms3),
                     "unit": "tokens/s", "gpu_launches": int(l3), "clocks": clk3, "roofline": roof3}
        del _p3, _s3
        torch.cuda.empty_cache()

    # ---- end to end through the C ABI with host buffers: every step uploads its inputs from pinned
    # host memory and downloads its results; two device problems take turns, so that the bus
    # carries one step's copies (both directions at once) while another step computes
    e2e = None
    if not args.no_e2e:
        pipe = runner.HostPipeline(w, slots=2, device=dev)
        h_in, h_out = pipe.pinned_inputs(), pipe.pinned_outputs()
        e2e_steps = max(4, min(args.steps, 10))
        for _ in range(3):
            pipe.submit(h_in, h_out)
        pipe.drain()
        barrier()
        e0.record()
        pipe.fence()
        for _ in range(e2e_steps):
            pipe.submit(h_in, h_out)
        pipe.fence()
        e1.record()
        barrier()
        e2e_ms = max_over_ranks(e0.elapsed_time(e1) / e2e_steps)
        nb = lambda t: t.numel() * t.element_size()  # noqa: E731
        e2e = {"value": world * w.tokens / (e2e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": sum(nb(t) for t in h_in.values()),
               "d2h_bytes_per_step": sum(nb(t) for t in h_out.values()),
               "pipeline": "2 device slots, upload / compute / download streams"}
        st_words = [int(x) for x in pipe.slots[0].workspace[:4].cpu().numpy().view("int32")[:1]]
        assert st_words[0] == 0, f"device status {st_words}"
        del pipe

    # ---- the oracle on the host cores (rank 0, N = 1 only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        ws = oracle_sample(w, SAMPLE_BATCH[args.config])
        sec = time_oracle(ws)
        cpu = {"value": ws.tokens / sec, "unit": "tokens/s", "cores": min(oracle.threads(), ws.B * ws.H),
               "kind": "oracle", "sample": f"{ws.name}: one fwd+bwd incl. selection, {sec:.1f} s"}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.dtype == "bf16" else "f32",
                "data": "synthetic", "config": cfg_desc, "clocks": clocks, "e2e": e2e,
                "gpu_launches": int(launches), "roofline": roof, "cpu_baseline": cpu,
                "graph_replay": graph_info, "secondary": secondary}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
