#!/usr/bin/env python
"""Benchmark of the blockwise-parallel-decoding hot path on B200.

One *step* is one complete decode of the headline workload (big model,
d_model 1024, k = 8, batch 1, 128 tokens) under controlled acceptance: every
merged score-and-propose iteration runs the decoder pass over the k block
positions, the k heads, the fused vocabulary top-1, verification and the cache
commit.  `value` is decoded tokens/s with everything resident on the device;
`e2e` goes through the public calls with host buffers (source ids in, token ids
out, encoder included).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
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

from bpd_inputs import WORKLOADS, forced_tail, geometric_schedule, make_source, make_weights  # noqa: E402

METRIC = "decoded tokens/s at batch 1 (d=1024, k=8)"
HEADLINE = "C3"
MEAN_ACCEPT = 5.0            # geometric mean of the controlled-acceptance schedule for the headline line
NOMINAL_HBM_GBS = 8000.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu capture
# summarised under profiles/ (None until a capture of the current kernel exists)
TRAFFIC = {"C3": 538161152 + 3223296}     # profiles/head_output_gemm_tc_c3.txt
TRAFFIC_LAYERS = {"C3": 178907648 + 4899328}   # profiles/layer_stack_kernel_c3.txt
# both lazy stages of the head output layers, per pass (profiles/projection_kernels_c4_batch32_tensor_pipe.txt)
TRAFFIC_PAIR = {"C4": int((138.4 + 3.7 + 844.4 + 3.2) * 1e6)}


def _peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, kind) from the driver-written measurement, else the machine's fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return float(p["hbm_gbs"]), float(p.get("bf16_tflops_sustained", 1400.0)), "measured"
    return 6650.0, 1400.0, "fallback"


DESCRIPTIONS = {
    "C2": "C2: base enc-dec 6+6, d_model 512, 8 heads, FFN 2048, vocab 32768, k=4 dense heads, batch 1, source 32 ids",
    "C3": "C3: big enc-dec 6+6, d_model 1024, 16 heads, FFN 4096, vocab 32768, k=8 dense heads, batch 1, source 40 ids",
    "C4": "C4: big enc-dec 6+6, d_model 1024, k=10 dense heads, batch 32, source lengths uniform in [10,80]",
    "C5": "C5: super-resolution shape, 6+6, d_model 512, vocab 256, k=10 dense heads, batch 1, 192 source ids",
    "C5L": "C5L: C5 with 1D local self-attention in the decoder (query blocks of 256, memory 256)",
}


def iteration_bytes(cfg, k, batch, mean_T, mean_S):
    """Bytes one merged iteration must move: every weight once, the cache once."""
    e = cfg.elem_bytes
    d, f, V, L, fh, km = cfg.d_model, cfg.d_ff, cfg.vocab, cfg.n_dec, cfg.d_hidden, cfg.k_model
    layers = L * (4 * d * d + 2 * d * d + 2 * d * f)
    w1 = d * km * fh if cfg.head_layout == 0 else d * k * fh
    w2 = k * d * km * fh if cfg.head_layout == 0 else k * d * fh
    return e * (layers + w1 + w2 + V * d) + batch * L * 2 * e * d * (mean_T + mean_S), e * w2


def max_over_ranks(ms: float, device=None) -> float:
    """Slowest rank's time (every rank must call it); identity without a process group."""
    import torch
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        t = torch.tensor([ms], device=device or "cpu", dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())
    return ms


def whole_job_tokens_per_s(tokens_per_rank: int, world: int, ms_step: float) -> float:
    """Replicas only: every rank decodes its own copy of the workload, no data-path collective;
    the job's throughput is all ranks' tokens over the slowest rank's time."""
    return world * tokens_per_rank / (ms_step * 1e-3)


def build_plan(w, greedy_ids, k, mean):
    plan = np.zeros((w.batch, w.n_decode, k - 1), dtype=np.int32)
    khats = []
    for b in range(w.batch):
        G, R = geometric_schedule(w.accept_seed * 1000 + b, mean, w.n_decode + 1)
        for j in range(w.n_decode):
            plan[b, j] = forced_tail(greedy_ids[b], j, k, int(G[j]), int(R[j]), w.cfg.vocab)
        j = 0
        while j < w.n_decode:
            kh = min(k, int(G[j]), w.n_decode - j)
            khats.append(kh)
            j += kh
    return plan, khats


class ClockSampler:
    """nvidia-smi clock / throttle samples while the timed region runs.  The GPU is named by its UUID
    (nvidia-smi numbers physical GPUs and ignores CUDA_VISIBLE_DEVICES, so a CUDA ordinal could
    describe somebody else's GPU); the id is recorded beside the samples."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id):
        self.index, self.rows, self.proc = str(gpu_id), [], None

    @staticmethod
    def identity(local: int) -> str:
        """UUID of CUDA device ``local`` of this process in nvidia-smi's spelling, else its PCI bus id."""
        import torch
        props = torch.cuda.get_device_properties(local)
        uuid = str(getattr(props, "uuid", "") or "")
        if uuid:
            return uuid if uuid.startswith("GPU-") else "GPU-" + uuid
        return f"{props.pci_domain_id:08x}:{props.pci_bus_id:02x}:{props.pci_device_id:02x}.0"

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            self.proc.wait()
            self.t.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "gpu": self.index}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "gpu": self.index}


# --------------------------------------------------------------------------- oracle legs (CPU)

def oracle_sample(w, blob, src, src_len, k, mean, n_tokens, repeats=1):
    """Time the oracle's merged blockwise decode (cached forward) on the first
    ``n_tokens`` tokens of row 0.  Returns (tokens/s, seconds per decode, threads)."""
    from oracle.decode import TransformerScorer, blockwise_merged, greedy
    from oracle.model import parse_blob
    om = parse_blob(blob)
    row = src[0, :src_len[0]]
    g = np.array(greedy(TransformerScorer(om, row, k=1, cached=True, capacity=n_tokens + 4), n_tokens).ids)
    G, R = geometric_schedule(w.accept_seed * 1000, mean, n_tokens + 1)
    times = []
    for _ in range(repeats):
        t0 = time.perf_counter()
        sc = TransformerScorer(om, row, k=k, cached=True, capacity=n_tokens + 2 * k + 2)
        res = blockwise_merged(sc, k, n_tokens,
                               tail_fn=lambda j, it: forced_tail(g, j, k, int(G[j]), int(R[j]), w.cfg.vocab))
        times.append(time.perf_counter() - t0)
        assert res.ids == list(g)
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    return n_tokens / float(np.mean(times)), times, threads


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WORKLOADS[HEADLINE]
    k = w.cfg.k_model
    blob = make_weights(w.cfg, w.weight_seed, w.sigma)
    src, src_len = make_source(w)
    n_tokens = w.n_decode                     # the whole decode: the same configuration as the GPU arm's step
    if int(os.environ.get("WORLD_SIZE", "1")) > 1:
        # torch's launcher pins OMP_NUM_THREADS to 1 for its children; rank 0 is the only rank that works here,
        # so it takes the host cores it would have had when started alone
        try:
            from threadpoolctl import threadpool_limits
            threadpool_limits(limits=len(os.sched_getaffinity(0)))
        except Exception:
            pass
    tps, times, threads = oracle_sample(w, blob, src, src_len, k, MEAN_ACCEPT, n_tokens,
                                        repeats=args.steps + args.warmup)
    timed = times[args.warmup:]
    value = n_tokens / float(np.mean(timed))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(np.mean(timed)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{DESCRIPTIONS[HEADLINE]}, decode {n_tokens} tokens, controlled acceptance "
                               f"(geometric mean {MEAN_ACCEPT})"},
        "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": threads, "kind": "oracle",
                         "arithmetic": "numpy float64, matrix products on the BLAS thread pool",
                         "sample": f"all {n_tokens} tokens of one decode per step"},
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# --------------------------------------------------------------------------- GPU arm

def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_1811_03115_b200.build import build_library
    build_library()
    import paper_1811_03115_b200 as bpd

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s)")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py times the CUDA path and needs a GPU; there is no CPU fallback "
                         "(--impl reference times the oracle)")
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local}"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"

    w = WORKLOADS[args.workload]
    cfg, k, N = w.cfg, w.cfg.k_model, w.n_decode
    blob = make_weights(cfg, w.weight_seed, w.sigma)
    src, src_len = make_source(w)
    model = bpd.Model(blob, dev)
    sess = bpd.Session(model, w.batch, w.max_src, N)
    sess.bpd_encode(src, src_len)
    g_ids, _, g_st = sess.bpd_decode_greedy(N)
    plan, khats = build_plan(w, g_ids, k, MEAN_ACCEPT)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_decodes(n_steps, mode):
        """Device-resident: state rewound on the device, results left on the device."""
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        ev0.record(sess.stream)
        for _ in range(n_steps):
            sess.bpd_rewind()
            if mode == "greedy":
                sess.bpd_decode_greedy(N, fetch=False)
            else:
                sess.bpd_decode_blockwise(k, N, fetch=False)
        ev1.record(sess.stream)
        barrier()
        return ev0.elapsed_time(ev1) / n_steps      # ms per decode

    # ---- headline: controlled acceptance, device resident
    sess.bpd_encode(src, src_len)
    sess.bpd_set_forced_plan(plan, k)
    timed_decodes(args.warmup, "block")
    launches0 = bpd.bpd_kernel_launches()
    with ClockSampler(ClockSampler.identity(local)) as clocks:
        ms_step = max_over_ranks(timed_decodes(args.steps, "block"), dev)
        launches = bpd.bpd_kernel_launches() - launches0
        # the timed region is a fraction of a second: keep the same load running (untimed) until nvidia-smi has
        # delivered a few samples, so that the clock record describes the GPU under this very workload
        # (the same count on every rank: ms_step is already the maximum over ranks)
        for _ in range(int(min(200, max(1, 600.0 / max(ms_step, 1e-3) / max(1, args.steps))))):
            timed_decodes(args.steps, "block")
    ids, _, st = sess.bpd_fetch_output(N)
    assert np.array_equal(ids, g_ids), "controlled-acceptance decode differs from greedy"
    assert st.row_iterations == len(khats)
    iters = st.iterations
    us_iter = 1e3 * ms_step / iters
    value = whole_job_tokens_per_s(w.batch * N, world, ms_step)

    # ---- per-phase timing of the same decode (events inside the pass), for the roofline of the dominant kernel
    sess.bpd_profile(True)
    timed_decodes(max(1, min(args.steps, 5)), "block")
    phases = [sess.bpd_profile_read(p) for p in range(4)]
    peak, peak_tf, peak_kind = _peaks()
    mean_T = 1 + N / 2.0
    it_bytes, w2_bytes = iteration_bytes(cfg, k, w.batch, mean_T, float(src_len.mean()))
    n_w2, ms_w2 = phases[2]
    # the priming pass evaluates the same k heads on one row per sequence: same weight bytes per launch
    w2_us = 1e3 * ms_w2 / max(1, n_w2)
    roofline_head_output = None
    if w.batch < 16:
        achieved = w2_bytes / (w2_us * 1e-6) / 1e9
        roofline = {"bound": "hbm", "kernel": "head output layers (k*d_model x k*d_hidden weights, + residual)",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_kind": f"of {peak_kind}", "traffic": TRAFFIC.get(args.workload),
                    "bytes_per_launch": w2_bytes, "us_per_launch": w2_us, "launches_timed": n_w2}
        if sess.layer_path == 2:
            # the whole decoder-layer stack is one launch here and the longest kernel of the pass: it is the one the
            # roofline line reports (bytes it must move: every layer's weights once, the cache once); the head output
            # projection, the kernel that moves most of the pass's bytes, keeps a line of its own
            roofline_head_output = roofline
            e = cfg.elem_bytes
            layer_bytes = e * cfg.n_dec * (6 * cfg.d_model * cfg.d_model + 2 * cfg.d_model * cfg.d_ff) + \
                w.batch * cfg.n_dec * 2 * e * cfg.d_model * (mean_T + float(src_len.mean()))
            n_l, ms_l = phases[0]
            l_us = 1e3 * ms_l / max(1, n_l)
            achieved = layer_bytes / (l_us * 1e-6) / 1e9
            roofline = {"bound": "hbm", "kernel": "decoder layer stack (persistent kernel: embedding, 6 layers, final layer norm)",
                        "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                        "peak_kind": f"of {peak_kind}", "traffic": TRAFFIC_LAYERS.get(args.workload),
                        "bytes_per_launch": layer_bytes, "us_per_launch": l_us, "launches_timed": n_l,
                        "note": "latency-bound: a chain of 19 dependent reductions across all SMs and 42 exchanges inside the clusters"}
    else:
        # batched: the same kernel is a dense contraction.  Sessions this wide evaluate the heads lazily: one launch
        # for head 1 at all batch*k positions, one for all k heads at the accepted position of each row; the
        # algorithmic flops are those of the two launches, the time is what the pair takes per pass (the priming
        # pass, one launch on batch rows, is left in the average)
        kf = cfg.k_model * cfg.d_hidden
        flops = 2.0 * (w.batch * k) * cfg.d_model * kf + 2.0 * w.batch * (k * cfg.d_model) * kf
        n_pass = max(1, phases[0][0])
        pair_us = 1e3 * ms_w2 / n_pass
        achieved = flops / (pair_us * 1e-6) / 1e12
        roofline = {"bound": "tensor", "kernel": "head output layers, both lazy stages (k*d_model x k*d_hidden weights)",
                    "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved / peak_tf,
                    "peak_kind": f"of {peak_kind} (sustained bf16)", "traffic": TRAFFIC_PAIR.get(args.workload),
                    "flops_per_pass": flops, "us_per_pass": pair_us, "launches_timed": n_w2}
    phase_us = {name: (1e3 * ms / max(1, n)) for name, (n, ms) in
                zip(["layers", "head_hidden", "head_output", "vocab_top1"], phases)}
    kernel_names = ["embed", "layer_norm", "qkv", "self_attn", "o_proj", "cross_q", "cross_attn", "cross_o",
                    "ffn1", "ffn2", "verify"]
    kernel_us = {}
    for i, name in enumerate(kernel_names):
        n, ms = sess.bpd_profile_read(4 + i)
        if n:
            kernel_us[name] = {"launches_per_pass": n / max(1, phases[0][0]), "us_per_launch": 1e3 * ms / n}
    sess.bpd_profile(False)

    # ---- other modes (context): greedy, free-running blockwise, mean-2 acceptance
    extra = {}
    if rank == 0 and not args.quick:
        sess.bpd_encode(src, src_len)
        timed_decodes(1, "greedy")
        ms_g = timed_decodes(max(1, args.steps // 2), "greedy")
        extra["greedy"] = {"tokens_per_s": w.batch * N / (ms_g * 1e-3), "us_per_pass": 1e3 * ms_g / N}
        sess.bpd_encode(src, src_len)
        timed_decodes(1, "block")
        ms_f = timed_decodes(max(1, args.steps // 2), "block")
        _, _, st_f = sess.bpd_fetch_output(N)
        extra["blockwise_free"] = {"tokens_per_s": w.batch * N / (ms_f * 1e-3),
                                   "us_per_iteration": 1e3 * ms_f / st_f.iterations,
                                   "mean_block": st_f.mean_block}
        plan2, kh2 = build_plan(w, g_ids, k, 2.0)
        sess.bpd_encode(src, src_len)
        sess.bpd_set_forced_plan(plan2, k)
        timed_decodes(1, "block")
        ms_2 = timed_decodes(max(1, args.steps // 2), "block")
        _, _, st_2 = sess.bpd_fetch_output(N)
        extra["controlled_mean2"] = {"tokens_per_s": w.batch * N / (ms_2 * 1e-3),
                                     "us_per_iteration": 1e3 * ms_2 / st_2.iterations,
                                     "mean_block": w.batch * N / len(kh2)}

    # ---- end to end through the public calls with host buffers
    sess.bpd_encode(src, src_len)
    e2e_times = []
    for i in range(args.warmup + args.steps):
        barrier()
        t0 = time.perf_counter()
        sess.bpd_encode(src, src_len)                 # H2D of the source ids + encoder
        sess.bpd_set_forced_plan(plan, k)             # H2D of the acceptance plan
        out_ids, out_len, _ = sess.bpd_decode_blockwise(k, N)   # D2H of the token ids
        torch.cuda.synchronize()
        e2e_times.append(time.perf_counter() - t0)
    e2e_ms = max_over_ranks(1e3 * float(np.mean(e2e_times[args.warmup:])), dev)
    h2d = src.nbytes + src_len.nbytes + plan.nbytes
    d2h = w.batch * N * 4 + w.batch * 4 + (3 + 17) * 8

    if rank != 0:
        return
    # ---- oracle on the host cores, bounded sample
    cpu = None
    if not args.no_cpu:
        n_tok = N
        tps, times, threads = oracle_sample(w, blob, src, src_len, k, MEAN_ACCEPT, n_tok, repeats=2)
        cpu = {"value": tps, "unit": "tokens/s", "cores": threads, "kind": "oracle",
               "arithmetic": "numpy float64, matrix products on the BLAS thread pool",
               "sample": f"row 0, all {n_tok} tokens of the decode, 2 decodes, {np.mean(times):.1f} s each"}
    line = {
        "metric": METRIC if args.workload == HEADLINE else f"decoded tokens/s ({args.workload})",
        "value": value, "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{DESCRIPTIONS[args.workload]}, decode {N} tokens, controlled acceptance "
                               f"(geometric mean {MEAN_ACCEPT}, mean accepted block {w.batch * N / len(khats):.2f})",
                   "l2": f"weights streamed per iteration ({it_bytes / 1e6:.0f} MB) "
                         + ("exceed L2; no flush needed" if it_bytes > 126e6 else "fit in L2: numbers are L2-warm"),
                   "replicas": world},
        "us_per_iteration": us_iter, "iterations_per_step": iters,
        "iteration_hbm_gbs": it_bytes / (us_iter * 1e-6) / 1e9,
        "iteration_frac_of_8tbs": it_bytes / (us_iter * 1e-6) / 1e9 / NOMINAL_HBM_GBS,
        "iteration_frac_of_measured": it_bytes / (us_iter * 1e-6) / 1e9 / peak,
        "phase_us": phase_us, "kernel_us_eager": kernel_us, "modes": extra,
        "clocks": clocks.summary(),
        "e2e": {"value": whole_job_tokens_per_s(w.batch * N, world, e2e_ms), "unit": "tokens/s", "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h)},
        "gpu_launches": int(launches),
        "roofline": roofline,
        "roofline_head_output": roofline_head_output,
        "layer_path": sess.layer_path,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def spawn_replicas(n: int, argv) -> int:
    """Start ``n`` copies of this script, one process per GPU, under torch's launcher and return its exit
    code.  The replicas share nothing on the data path; the process group serves the barrier around the
    timed region and the maximum over ranks."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__), *argv]
    return subprocess.call(cmd)


def main(argv=None):
    argv = list(sys.argv[1:] if argv is None else argv)
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=sorted(DESCRIPTIONS), help="configuration to time")
    ap.add_argument("--quick", action="store_true", help="skip the context modes")
    ap.add_argument("--no-cpu", action="store_true", help="skip the oracle leg")
    args = ap.parse_args(argv)
    if args.gpus < 1:
        ap.error("--gpus must be at least 1")
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand rather than by a launcher: become the launcher of N replicas
        sys.exit(spawn_replicas(args.gpus, argv))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
