#!/usr/bin/env python
"""Benchmark of one DiT-block attention (`sol_attn3d_forward`) on synthetic inputs.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload highres] [--impl ours|reference]

A step is one pass of the whole hot path (key-validity bits when needed, rotary
prologue, attention kernel) over one batch.  Prints ONE JSON line.  For N > 1
(torchrun) every rank runs an independent replica of the same workload: the
path has no exchange step, so there is no collective on the data path.

``--impl reference`` times the fp64 CPU oracle on a bounded sample of the same
workload on the host cores (rank 0 only).
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2609_35110_b200 import workloads as wl  # noqa: E402

METRIC = "attention_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16 = 2250.0
TRAFFIC_SUMMARY = os.path.join(ROOT, "profiles", "attn_fwd_kernel_dram_traffic.md")
SM_COUNT = 148
TENSOR_FLOP_PER_CLK_PER_SM = 8192       # dense bf16 on one SM's tensor core


def load_ncu_traffic(workload):
    """dram__bytes_read.sum + dram__bytes_write.sum of one attention-kernel launch, as recorded in the tracked ncu
    summary of that capture (lines `traffic <workload>: dram_read_bytes=R dram_write_bytes=W`).  None if absent."""
    try:
        with open(TRAFFIC_SUMMARY) as f:
            for line in f:
                parts = line.strip().strip("`").split()
                if len(parts) >= 4 and parts[0] == "traffic" and parts[1].rstrip(":") == workload:
                    kv = dict(x.split("=", 1) for x in parts[2:] if "=" in x)
                    return int(kv["dram_read_bytes"]) + int(kv["dram_write_bytes"]), \
                        "ncu capture of this workload (one pass, two DRAM counters), profiles/attn_fwd_kernel_dram_traffic.md"
    except (OSError, KeyError, ValueError):
        pass
    return None, None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"burst": float(d["bf16_tflops"]), "sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS, "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(pw) if pw else None, "samples": len(sm), "reasons": sorted(reasons)}


def max_over_ranks(values, dist=None, device="cpu"):
    """Element-wise maximum of a list of per-rank times over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def whole_job_tflops(flops_per_replica, world, ms_per_step):
    """Replicas only: every rank runs the same workload, the job's rate is world x one replica's work over the slowest time."""
    return world * flops_per_replica / (ms_per_step * 1e-3) / 1e12


def oracle_sample(w, inp_cpu, heads_sample, rows_per_head):
    """(seq, head, rows) selection used by the CPU baseline: the parity rows of a few heads."""
    sel = []
    for s in range(w.n_seqs):
        for h in heads_sample:
            rows = wl.sample_rows(w, s, h, rows_per_head)
            sel.append((s, h, torch.from_numpy(rows)))
    return sel


def sample_flops(w, sel):
    fl = 0.0
    for (s, h, rows) in sel:
        nk = w.seqs[s].n_tokens
        if w.valid_text is not None:
            nk -= w.seqs[s].text_len - w.valid_text[s]
        fl += 4.0 * len(rows) * nk * w.head_dim
    return fl


def run_oracle(w, inp_cpu, sel, q_gain=None, k_gain=None):
    from oracle import attn3d_oracle as orc   # CPU-baseline leg: the one place bench.py runs the oracle
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    t0 = time.perf_counter()
    ref = orc.attn3d_oracle(inp_cpu.q, inp_cpu.k, inp_cpu.v, seqs, w.rope_dims, w.theta, inp_cpu.key_mask, sel,
                            q_gain=q_gain, k_gain=k_gain)
    return ref, time.perf_counter() - t0


def cpu_sample_spec(w, scale=1.0):
    """How much oracle work to time: about 10-30 s on a 16-core host."""
    if w.name == "tiny":
        return list(range(w.heads)), 0
    n_heads = {"lowres": 40, "highres": 18, "cfg_batch": 9, "varlen": 18}.get(w.name, 2)
    n_heads = max(1, min(w.heads, int(round(n_heads * scale))))
    step = max(1, w.heads // n_heads)
    return list(range(0, w.heads, step))[:n_heads], (w.rows_per_head or 0)


def exchange_bench(args, w, dev, B, peaks, config):
    """One rank's share of a G-way sequence-parallel exchange around the attention: the layout / quantisation
    kernels and the head-sharded attention, each timed alone with CUDA events (best and mean of `steps`)."""
    G = args.exchange
    heads, D, total = w.heads, w.head_dim, w.total_tokens
    if heads % G or G > B.MAX_RANKS:
        raise SystemExit(f"--exchange {G}: heads ({heads}) must be divisible and G <= {B.MAX_RANKS}")
    hl = heads // G
    n_local = -(-total // G)
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    packed = torch.randn((n_local, 3, heads, D), generator=gen, device=dev).to(torch.bfloat16)   # packed QKV storage
    q, k, v = packed[:, 0], packed[:, 1], packed[:, 2]
    send = torch.empty((G, n_local, 3, hl, D), dtype=torch.bfloat16, device=dev)
    rb_in = B.sol_attn3d_exchange_record_bytes(B.WIRE_QKV_INT8, D)
    rb_out = B.sol_attn3d_exchange_record_bytes(B.WIRE_OUT_INT8, D)
    send8 = torch.empty((G, n_local, hl, rb_in), dtype=torch.uint8, device=dev)
    qkv = torch.randn((total, 3, hl, D), generator=gen, device=dev).to(torch.bfloat16)
    v_scratch = torch.empty((total, hl, D), dtype=torch.bfloat16, device=dev)
    qkv_unpacked = torch.empty_like(qkv)     # the unpack kernel's own output: the attention below keeps its N(0,1) inputs
    rec_in = torch.empty((total, hl, rb_in), device=dev, dtype=torch.uint8)
    # realistic records: the N(0,1) QKV shard as a sender would have quantised it
    B.sol_attn3d_exchange_pack_qkv_int8(qkv[:, 0], qkv[:, 1], qkv[:, 2], 1, [rec_in.data_ptr()], 0)
    shard = (0.1 * torch.randn((total, hl, D), generator=gen, device=dev)).to(torch.bfloat16)
    shard8 = torch.empty((total, hl, D), dtype=torch.uint8, device=dev)
    rec_out = torch.empty((total, hl, rb_out), dtype=torch.uint8, device=dev)
    recv = torch.randn((G, n_local, hl, D), generator=gen, device=dev).to(torch.bfloat16)
    recv_rec = torch.randint(1, 120, (n_local, heads, rb_out), generator=gen, device=dev, dtype=torch.uint8)
    merged = torch.empty((n_local, heads, D), dtype=torch.bfloat16, device=dev)
    st = (3 * hl * D, D)
    seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
    attn = B.Attn3d(seqs, hl, D, w.rope_dims, w.theta, dev, q_strides=st, k_strides=st, v_strides=st)
    per = -(-total // G)
    tok_begin = [min(g * per, total) for g in range(G)] + [total]
    owners = [torch.empty((max(tok_begin[g + 1] - tok_begin[g], 1), heads, D), dtype=torch.bfloat16, device=dev) for g in range(G)]
    sptr = [send[g].data_ptr() for g in range(G)]
    sptr8 = [send8[g].data_ptr() for g in range(G)]
    bf = 2
    kernels = {
        # name: (callable, bytes read + written)
        "pack_qkv": (lambda: B.sol_attn3d_exchange_pack_qkv(q, k, v, G, sptr, 0), 2 * packed.numel() * bf),
        "merge_heads_bf16": (lambda: B.sol_attn3d_exchange_merge_heads(recv, merged, n_local, heads, D * bf, G), 2 * recv.numel() * bf),
        "pack_qkv_int8": (lambda: B.sol_attn3d_exchange_pack_qkv_int8(q, k, v, G, sptr8, 0), packed.numel() * bf + send8.numel()),
        "unpack_qkv_int8": (lambda: B.sol_attn3d_exchange_unpack_qkv_int8(rec_in, qkv_unpacked, total, hl, D),
                            rec_in.numel() + qkv.numel() * bf),
        "quantize_out_int8": (lambda: B.sol_attn3d_exchange_quantize_out_int8(shard, rec_out), shard.numel() * bf + rec_out.numel()),
        "dequantize_out_int8": (lambda: B.sol_attn3d_exchange_dequantize_out_int8(recv_rec, merged), recv_rec.numel() + merged.numel() * bf),
        "attention_shard_bf16": (lambda: B.sol_attn3d_forward(attn.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], shard, None), None),
        "attention_shard_e4m3": (lambda: B.sol_attn3d_forward_e4m3(attn.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], shard8, None), None),
        # the wire formats fused into the neighbours (Section 3.3): INT8 records written by the attention epilogue, and
        # the attention fed by INT8 QKV records (dequantised inside the rotary producer)
        "attention_shard_int8_out": (lambda: B.sol_attn3d_forward_int8(attn.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], rec_out, None), None),
        "attention_shard_from_int8_records": (lambda: B.sol_attn3d_forward_qkv_int8(attn.plan, rec_in, v_scratch, shard, None), None),
        "attention_shard_scatter": (lambda: B.sol_attn3d_forward_scatter(attn.plan, qkv[:, 0], qkv[:, 1], qkv[:, 2], None,
                                                                         [o.data_ptr() for o in owners], tok_begin, heads, 0), None),
    }
    if args.exchange_kernel != "all":
        kernels = {args.exchange_kernel: kernels[args.exchange_kernel]}
    hbm = peaks.get("hbm_gbs") if isinstance(peaks, dict) else None
    shard_flops = w.flops() / G
    res = {}
    for name, (fn, nbytes) in kernels.items():
        for _ in range(max(3, args.warmup)):
            fn()
        torch.cuda.synchronize()
        ts = []
        for _ in range(args.steps):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        ms = sum(ts) / len(ts)
        r = {"ms": ms, "ms_best": min(ts)}
        if nbytes is not None:
            r["bytes"] = nbytes
            r["gbps"] = nbytes / ms / 1e6
            if hbm:
                r["frac_of_measured_hbm"] = r["gbps"] / hbm
        else:
            r["tflops"] = shard_flops / ms / 1e9
        res[name] = r
    assert attn.status() == 0
    print(json.dumps({"metric": "exchange_kernels_ms", "unit": "ms", "n_gpus": 1, "steps": args.steps,
                      "warmup": max(3, args.warmup), "exchange_ranks": G, "tokens_per_rank": n_local, "heads_per_rank": hl,
                      "hbm_peak_gbs": hbm, "config": config, "data": "synthetic", "kernels": res}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="highres", choices=wl.CONFIG_ORDER)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--sparse-tau", type=float, default=None,
                    help="time sol_attn3d_forward_sparse with this tau (block-sparse variant of Section 3.4)")
    ap.add_argument("--qknorm", action="store_true",
                    help="time sol_attn3d_forward_qknorm (QK RMS-norm fused into the rotary producer) instead")
    ap.add_argument("--exchange", type=int, default=0, metavar="G",
                    help="instead of the forward: time one rank's kernels of a G-way sequence-parallel exchange "
                         "(Section 3.2) at the workload's shape and print their ms and GB/s")
    ap.add_argument("--exchange-kernel", default="all",
                    help="with --exchange: run only this kernel (e.g. for a profiler capture)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    w = wl.CONFIGS[args.workload]
    config = {"workload": f"{w.name}: " + ", ".join(f"[{s.text_len} text + {s.T}x{s.H}x{s.W}]" for s in w.seqs)
              + f", heads={w.heads}, head_dim={w.head_dim}, rope={list(w.rope_dims)}",
              "tokens": w.total_tokens, "flops_per_step": w.flops(), "replicas": world,
              "l2_policy": "inputs (%.2f GB) exceed L2" % (w.algorithmic_bytes() / 1e9)}
    peaks = load_peaks()

    # ------------------------------------------------------------------ reference arm = the oracle
    if args.impl == "reference":
        if rank != 0:
            return 0
        inp = wl.make_inputs(w, "cpu")
        heads_s, rows = cpu_sample_spec(w, scale=0.34)
        sel = oracle_sample(w, inp, heads_s, rows)
        fl = sample_flops(w, sel)
        # the oracle has no state to warm beyond the allocator and the BLAS threads: one untimed pass over one group
        warm_done = 1 if args.warmup > 0 else 0
        for _ in range(warm_done):
            run_oracle(w, inp, sel[:1])
        times = []
        for _ in range(args.steps):
            _, dt = run_oracle(w, inp, sel)
            times.append(dt)
        dt = sum(times) / len(times)
        val = fl / dt / 1e12
        sample = f"{len(sel)} (seq, head) groups x {len(sel[0][2])} query rows against all keys"
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": warm_done, "warmup_note": "one untimed oracle pass over one (seq, head) group",
            "ms_per_step": dt * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": config,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}))
        return 0

    # ------------------------------------------------------------------ our arm
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the attention path has no CPU fallback")
    from paper_2609_35110_b200 import binding as B
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=dev)

    if args.exchange:
        return exchange_bench(args, w, dev, B, peaks, config)

    warmup = max(3, args.warmup)
    inp = wl.make_inputs(w, dev)
    attn = B.Attn3d.from_workload(w, dev)
    out = torch.empty((w.total_tokens, w.heads, w.head_dim), dtype=torch.bfloat16, device=dev)
    B.sol_attn3d_set_profiling(attn.plan, True)
    stream = torch.cuda.current_stream()
    if args.qknorm:
        # synthetic learned gains (the paper's checkpoints are not available)
        gg = torch.Generator(device=dev).manual_seed(w.seed + 77)
        q_gain = 1.0 + 0.1 * torch.randn(w.head_dim, generator=gg, device=dev, dtype=torch.float32)
        k_gain = 1.0 + 0.1 * torch.randn(w.head_dim, generator=gg, device=dev, dtype=torch.float32)
        config["qknorm"] = "RMS-norm over head_dim with synthetic gains, eps 1e-6, fused into the rotary producer"

        def forward(q, k, v, mask, out):
            B.sol_attn3d_forward_qknorm(attn.plan, q, k, v, out, mask, q_gain, k_gain, 1e-6)
    elif args.sparse_tau is not None:
        q_gain = k_gain = None
        sparse_ws = torch.empty(B.sol_attn3d_sparse_workspace_bytes(attn.plan), dtype=torch.uint8, device=dev)
        config["sparse"] = f"block-sparse, tau={args.sparse_tau}, query blocks 256 x KV blocks 128"

        def forward(q, k, v, mask, out):
            B.sol_attn3d_forward_sparse(attn.plan, q, k, v, out, mask, args.sparse_tau, sparse_ws)
    else:
        q_gain = k_gain = None

        def forward(q, k, v, mask, out):
            attn.forward(q, k, v, mask, out=out)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warmup):
        forward(inp.q, inp.k, inp.v, inp.key_mask, out)
    torch.cuda.synchronize()
    if attn.status() != 0:
        raise SystemExit("device reported a wait time-out during warm-up")

    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else
                           int(os.environ["CUDA_VISIBLE_DEVICES"].split(",")[local_rank]))
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    kernel_ms = []
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        forward(inp.q, inp.k, inp.v, inp.key_mask, out)
    ev1.record(stream)
    barrier()
    total_ms = ev0.elapsed_time(ev1)
    clocks = sampler.stop() if rank == 0 else None
    # kernels enqueued by one forward of the timed loop, as counted by the library while it launched them
    launches = B.sol_attn3d_last_launch_count(attn.plan)

    # per-kernel durations (CUDA events recorded by the library on the launching stream): a second
    # short loop so that the blocking event read never sits inside the timed region above
    for _ in range(min(args.steps, 5)):
        forward(inp.q, inp.k, inp.v, inp.key_mask, out)
        kernel_ms.append(B.sol_attn3d_last_forward_ms(attn.plan))
    torch.cuda.synchronize()
    if attn.status() != 0:
        raise SystemExit("device reported a wait time-out")

    # ------------------------------------------------------------------ end to end (host buffers)
    e2e = None
    if not args.no_e2e:
        hq, hk, hv = (t.cpu().pin_memory() for t in (inp.q, inp.k, inp.v))
        hmask = None if inp.key_mask is None else inp.key_mask.cpu().pin_memory()
        hout = torch.empty(out.shape, dtype=out.dtype).pin_memory()
        dq, dk, dv = (torch.empty_like(t) for t in (inp.q, inp.k, inp.v))
        dmask = None if inp.key_mask is None else torch.empty_like(inp.key_mask)
        e_steps = max(2, min(args.steps, 4))

        plain = not args.qknorm and args.sparse_tau is None
        staging = torch.empty(B.sol_attn3d_host_staging_bytes(attn.plan), dtype=torch.uint8, device=dev) if plain else None

        def e2e_step():
            if plain:
                # the library's own host-buffer entry point: copies of one head group overlap the kernels of another
                B.sol_attn3d_forward_host(attn.plan, hq, hk, hv, hout, hmask, staging, 0)
                return
            dq.copy_(hq, non_blocking=True)
            dk.copy_(hk, non_blocking=True)
            dv.copy_(hv, non_blocking=True)
            if dmask is not None:
                dmask.copy_(hmask, non_blocking=True)
            forward(dq, dk, dv, dmask, out)
            hout.copy_(out, non_blocking=True)

        e2e_step()
        barrier()
        ev0.record(stream)
        for _ in range(e_steps):
            e2e_step()
        ev1.record(stream)
        barrier()
        e_ms = ev0.elapsed_time(ev1) / e_steps
        h2d = 3 * inp.q.numel() * 2 + (0 if hmask is None else hmask.numel())
        e2e = {"ms": e_ms, "h2d": h2d, "d2h": out.numel() * 2, "steps": e_steps}
        e2e["api"] = "sol_attn3d_forward_host (head groups, copies overlapped)" if plain else "copies + forward + copy on one stream"
        if plain:
            torch.cuda.synchronize()
            e2e["max_abs_vs_device_forward"] = float((hout.to(dev).float() - out.float()).abs().max())
        del hq, hk, hv, hout, dq, dk, dv, staging

    # ------------------------------------------------------------------ max over ranks
    ms_per_step = total_ms / args.steps
    if dist is not None:
        ms_per_step, e_max = max_over_ranks([ms_per_step, e2e["ms"] if e2e else 0.0], dist, dev)
        if e2e:
            e2e["ms"] = e_max
    if rank != 0:
        if dist is not None:
            dist.barrier()
            dist.destroy_process_group()
        return 0

    flops = w.flops()                       # valid keys only: no credit for skipped work
    if args.sparse_tau is not None:
        sel_tiles, all_tiles = B.sol_attn3d_sparse_stats(attn.plan, sparse_ws)
        config["sparse_density"] = sel_tiles / max(all_tiles, 1)
        config["dense_equivalent_tflops"] = whole_job_tflops(flops, world, ms_per_step)
        flops *= sel_tiles / max(all_tiles, 1)          # executed (query block, key tile) pairs only
    value = whole_job_tflops(flops, world, ms_per_step)
    # Per-kernel CUDA-event times come from the short second loop (each step followed by a blocking read, so the GPU
    # idles between steps and runs a little faster there than inside the long timed region).  What the roofline line
    # uses is the attention kernel's share of those times applied to the timed region's own time per step.
    attn_ms_probe = statistics.mean(k[2] for k in kernel_ms)
    probe_sum = statistics.mean(k[0] + k[1] + k[2] for k in kernel_ms)
    attn_ms = ms_per_step * attn_ms_probe / probe_sum
    rope_ms = statistics.mean(k[1] for k in kernel_ms)
    bits_ms = statistics.mean(k[0] for k in kernel_ms)
    achieved = flops / (attn_ms * 1e-3) / 1e12
    long_step = total_ms > 1000.0
    peak = peaks["sustained"] if long_step else peaks["burst"]
    traffic, traffic_note = load_ncu_traffic(w.name)
    if args.sparse_tau is not None:         # the capture is of the dense launch; the sparse one was not captured
        traffic, traffic_note = None, "not captured for the block-sparse launch"
    # cycles of one attention launch at the SM clock sampled during the timed region: separates gains in the
    # dependency chain (fewer cycles) from gains in power (more MHz under the cap)
    sm_mhz = clocks.get("sm_mhz") if clocks else None
    attn_mcycles = attn_ms * 1e-3 * sm_mhz if sm_mhz else None
    per_clock = flops / (attn_mcycles * 1e6 * SM_COUNT * TENSOR_FLOP_PER_CLK_PER_SM) if attn_mcycles else None

    # ------------------------------------------------------------------ CPU baseline (oracle, bounded sample)
    cpu = None
    parity = None
    if not args.no_cpu_baseline and world == 1 and args.sparse_tau is not None:
        # block-sparse leg: the oracle on a few sampled (head, rows) groups, over the blocks the GPU selected
        from oracle import attn3d_oracle as orc
        seqs = [(s.text_len, s.T, s.H, s.W) for s in w.seqs]
        q_cpu, k_cpu, v_cpu = inp.q.cpu(), inp.k.cpu(), inp.v.cpu()
        mask_cpu = None if inp.key_mask is None else inp.key_mask.cpu()
        select, picked = [], []
        for h in sorted({0, w.heads - 1}):
            sq0 = w.seqs[0]
            nq, nk = (sq0.n_tokens + 255) // 256, (sq0.n_tokens + 127) // 128
            m = torch.zeros(nq, nk, dtype=torch.bool)
            for i in range(nq):
                m[i, B.sol_attn3d_sparse_selection(attn.plan, sparse_ws, 0, h, i, nk)] = True
            picked.append(m)
            select.append((0, h, torch.from_numpy(wl.sample_rows(w, 0, h, 96))))
        t0 = time.perf_counter()
        ref, _, _ = orc.attn3d_sparse_oracle(q_cpu, k_cpu, v_cpu, seqs, w.rope_dims, w.theta, args.sparse_tau, 256, 128,
                                             mask_cpu, selection=picked, select=select)
        dt = time.perf_counter() - t0
        o_cpu = out.cpu()
        got = torch.cat([o_cpu[rows_, h] for (_, h, rows_) in select])
        ma, rl = orc.compare(got, torch.cat(ref))
        kept = sum(float(m.float().mean()) for m in picked) / len(picked)
        fl = sum(4.0 * len(r_) * w.seqs[0].n_tokens * w.head_dim for (_, _, r_) in select) * kept
        cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": torch.get_num_threads(), "kind": "oracle", "seconds": dt,
               "sample": f"{len(select)} heads x 96 query rows of sequence 0 over the KV blocks the GPU selected (fp64); "
                         "the time includes rotating every token of those heads"}
        parity = {"max_abs": ma, "rel_l2": rl, "rows": int(got.shape[0]), "tol_max_abs": 2e-2, "tol_rel_l2": 5e-3,
                  "ok": bool(ma <= 2e-2 and rl <= 5e-3), "selection": "the GPU's own, read back per (head, query block)"}
    if not args.no_cpu_baseline and world == 1 and args.sparse_tau is None:
        from oracle import attn3d_oracle as orc
        inp_cpu = wl.Inputs(inp.q.cpu(), inp.k.cpu(), inp.v.cpu(), None if inp.key_mask is None else inp.key_mask.cpu())
        heads_s, rows = cpu_sample_spec(w)
        sel = oracle_sample(w, inp_cpu, heads_s, rows)
        ref, dt = run_oracle(w, inp_cpu, sel, None if q_gain is None else q_gain.cpu(),
                             None if k_gain is None else k_gain.cpu())
        cpu = {"value": sample_flops(w, sel) / dt / 1e12, "unit": UNIT, "cores": torch.get_num_threads(),
               "kind": "oracle", "seconds": dt,
               "sample": f"{len(sel)} (seq, head) groups x {len(sel[0][2])} query rows against all keys (fp64)"}
        # the same rows double as a full-size parity check of the timed configuration
        cu = w.cu_seqlens
        o_cpu = out.cpu()
        got = torch.cat([o_cpu[cu[s] + rows_, h] for (s, h, rows_) in sel])
        ma, rl = orc.compare(got, torch.cat(ref))
        parity = {"max_abs": ma, "rel_l2": rl, "rows": int(got.shape[0]), "tol_max_abs": 2e-2, "tol_rel_l2": 5e-3,
                  "ok": bool(ma <= 2e-2 and rl <= 5e-3)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": config,
        "pct_of_bf16_peak": {"measured_burst_%.1f" % peaks["burst"]: 100 * value / world / peaks["burst"],
                             "measured_sustained_%.1f" % peaks["sustained"]: 100 * value / world / peaks["sustained"],
                             "nominal_%.0f" % NOMINAL_BF16: 100 * value / world / NOMINAL_BF16},
        "kernel_ms": {"keybits": bits_ms, "rope_prologue": rope_ms, "attention": attn_ms_probe,
                      "attention_in_timed_region": attn_ms,
                      "note": "per-kernel events from a separate short loop; attention_in_timed_region = ms_per_step x the "
                              "attention's share of them, the duration the roofline line uses"},
        "attention_mcycles": attn_mcycles, "tensor_pipe_busy_per_clock": per_clock,
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "peak_kind": ("sustained" if long_step else "burst") + " bf16, " + peaks["source"],
                     "kernel": "attn_fwd_kernel<%d>" % w.head_dim, "traffic": traffic, "traffic_note": traffic_note,
                     "algorithmic_bytes": w.algorithmic_bytes(),
                     "frac_of_burst": achieved / peaks["burst"]},
        "clocks": clocks,
        "gpu_launches": launches * args.steps,
    }
    if e2e:
        line["e2e"] = {"value": whole_job_tflops(flops, world, e2e["ms"]), "unit": UNIT, "ms_per_step": e2e["ms"],
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"],
                       "api": e2e.get("api"), "max_abs_vs_device_forward": e2e.get("max_abs_vs_device_forward")}
    if cpu:
        line["cpu_baseline"] = cpu
    if parity:
        line["parity_vs_oracle"] = parity
    print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())
