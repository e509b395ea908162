#!/usr/bin/env python
"""Benchmark of the BitLinear forward (BitNet b1.58) on B200.

Headline workload: the 70B-shaped decode step -- all 80 x 7 BitLinear projections of the decoder at M = 1 token,
17.1 GB of 2-bit weights resident in HBM -- run through bitlinear_forward_sequence.  One "step" = activation
quantisation + ternary matmul + dequantisation for all 560 matrices.  Metric: packed-weight GB/s = (sum of N*K/4
bytes) / step time.  The 3B-shaped step (805 MB per step, where the fixed cost of a launch shows) is reported beside it
with its own roofline, end-to-end and CPU blocks; the prefill GEMM has a roofline block against the int8 tensor peak
measured in the same run.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-extras]

Prints one JSON line.  The K timed steps are repeated in rounds until at least a second has been timed; the line
reports the median round (and the fastest).  With --gpus N > 1 (under torchrun) every rank runs an independent
replica of the workload on its own GPU ("replicas only": the path needs no exchange) and the aggregate is reported.
--impl reference times the CPU oracle on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import re
import statistics
import subprocess
import sys
import tempfile
import time
from pathlib import Path

ROOT = Path(__file__).resolve().parent
sys.path.insert(0, str(ROOT))

METRIC = "decode BitLinear packed-weight GB/s"
UNIT = "GB/s"
WORKLOAD = "70b_decode"
MIN_TIMED_S = 1.0   # the timed rounds go on until this much device time has been measured
MAX_ROUNDS = 400


def ncu_traffic_ratio():
    """dram__bytes_read.sum + dram__bytes_write.sum per algorithmic byte of the streaming kernel, from the committed ncu
    summary -- or None when the kernel's source has changed since that capture (the summary records the source's hash).
    Traffic grows in proportion to the packed bytes, so the figure for a launch is the ratio times its packed bytes."""
    summary = ROOT / "profiles" / "decode_mma_kernel_7b_up_x48_M1.md"
    source = ROOT / "paper_2402_17764_b200" / "csrc" / "decode_gemv.cu"
    try:
        text = summary.read_text()
        ratio = re.search(r"traffic_ratio:\s*([0-9.]+)", text)
        sha = re.search(r"decode_gemv_sha256:\s*([0-9a-f]{64})", text)
        if not ratio or not sha or hashlib.sha256(source.read_bytes()).hexdigest() != sha.group(1):
            return None
        return float(ratio.group(1))
    except OSError:
        return None


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ---------------------------------------------------------------------------------------------------
# clocks

class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "50"], stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                smax.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        try:
            os.unlink(self.file.name)
        except OSError:
            pass
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = max(smax)
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------------------------------
# workloads (CUDA arm)

class Weights:
    """Resident packed weights (and their gammas) of a list of BitLinear matrices."""

    def __init__(self, layer_shapes, n_layers, copies=1, seed_base=0, trits=False):
        import torch
        from paper_2402_17764_b200 import binding as B
        from paper_2402_17764_b200 import synthetic as S
        self.trits = trits   # the base-3 format, five weights per byte
        nbytes = B.packed_bytes_trits if trits else B.packed_bytes
        quantize = B.quantize_weights_trits if trits else B.quantize_weights
        self.entries = [(li, mi, sh) for li in range(n_layers * copies) for mi, sh in enumerate(layer_shapes)]
        a256 = lambda n: (n + 255) // 256 * 256
        sizes = [a256(nbytes(sh.N, sh.K)) for _, _, sh in self.entries]
        self.packed_all = torch.empty(sum(sizes), dtype=torch.uint8, device="cuda")
        self.gammas = torch.empty(len(self.entries), dtype=torch.float32, device="cuda")
        self.packed, self.seeds = [], []
        self.algorithmic_bytes = 0   # of the 2-bit format (N K / 4), whatever the stored format
        self.stored_bytes = 0
        po = 0
        for i, (li, mi, sh) in enumerate(self.entries):
            seed = seed_base + li * 16 + mi
            W = S.latent_weights(sh.N, sh.K, seed, device="cuda")
            packed = self.packed_all[po:po + nbytes(sh.N, sh.K)]
            quantize(W, 1e-5, packed=packed, gamma=self.gammas[i:i + 1])
            del W
            self.packed.append(packed)
            self.seeds.append(seed)
            self.algorithmic_bytes += S.packed_weight_bytes(sh.N, sh.K)
            self.stored_bytes += nbytes(sh.N, sh.K)
            po += sizes[i]
        torch.cuda.synchronize()


class Stack:
    """The matrices of a Weights object with one contiguous X and one contiguous Y buffer for M tokens each."""

    def __init__(self, layer_shapes, n_layers, M, outlier_frac=0.0, outlier_scale=1.0, copies=1, seed_base=0, weights=None):
        import torch
        from paper_2402_17764_b200 import synthetic as S
        self.M = M
        self.weights = weights or Weights(layer_shapes, n_layers, copies, seed_base)
        entries = self.weights.entries
        a256 = lambda n: (n + 255) // 256 * 256
        x_sizes = [a256(M * sh.K * 2) // 2 for _, _, sh in entries]
        y_sizes = [a256(M * sh.N * 2) // 2 for _, _, sh in entries]
        self.X_all = torch.empty(sum(x_sizes), dtype=torch.bfloat16, device="cuda")
        self.Y_all = torch.zeros(sum(y_sizes), dtype=torch.bfloat16, device="cuda")
        self.layers = []
        self.algorithmic_bytes = self.weights.algorithmic_bytes
        self.int_ops = 0
        xo = yo = 0
        for i, (li, mi, sh) in enumerate(entries):
            X = self.X_all[xo:xo + M * sh.K].view(M, sh.K)
            X.copy_(S.activations(M, sh.K, self.weights.seeds[i], device="cuda", outlier_frac=outlier_frac,
                                  outlier_scale=outlier_scale))
            Y = self.Y_all[yo:yo + M * sh.N].view(M, sh.N)
            self.layers.append((self.weights.packed[i], self.weights.gammas[i:i + 1], X, Y, sh.N))
            self.int_ops += 2 * M * sh.N * sh.K
            xo += x_sizes[i]
            yo += y_sizes[i]
        torch.cuda.synchronize()


def time_sequence(stack, steps, warmup, dist_barrier=None, kernel_steps=None, min_timed_s=MIN_TIMED_S):
    """-> dict: ms per step as the median and the minimum over rounds of `steps` whole steps each (rounds are repeated
    until `min_timed_s` of device time has been measured), and ms per launch of the matmul kernel alone, from a further
    pass with events around that launch."""
    import torch
    from paper_2402_17764_b200 import binding as B
    seq = B.Sequence(stack.layers, trits=stack.weights.trits)
    for _ in range(warmup):
        seq.forward()
    rounds, total_ms = [], 0.0
    while True:
        torch.cuda.synchronize()
        if dist_barrier:
            dist_barrier()
        start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        start.record()
        for _ in range(steps):
            seq.forward()      # activation quantiser + persistent matmul (which may start early) for all matrices
        end.record()
        torch.cuda.synchronize()
        if dist_barrier:
            dist_barrier()
        ms = start.elapsed_time(end)
        rounds.append(ms / steps)
        total_ms += ms
        enough = total_ms >= min_timed_s * 1e3 or len(rounds) >= MAX_ROUNDS
        if dist_barrier:   # every rank must take the same number of rounds
            enough = all_ranks_agree(torch.distributed, enough, "cuda") or len(rounds) >= MAX_ROUNDS
        if enough:
            break
    status = B.poll_status(seq.workspace)
    if status != 0:
        raise RuntimeError(f"device status {status}")
    # the same steps again with events around the matmul launch (they keep the two launches apart)
    n = kernel_steps or max(5, min(steps, 200))
    mids = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
    for a, b in mids:
        seq.forward_stage(1)
        a.record()
        seq.forward_stage(2)
        b.record()
    torch.cuda.synchronize()
    kern = statistics.median(a.elapsed_time(b) for a, b in mids)
    seq.close()
    return {"ms": statistics.median(rounds), "ms_min": min(rounds), "rounds": len(rounds), "kernel_ms": kern,
            "timed_s": total_ms * 1e-3}


def time_e2e(stack, steps, warmup):
    """Host buffers in, host buffers out: per step one H2D copy of all X from pinned memory, the sequence, one D2H
    copy of all Y into pinned memory.  -> (ms per step with the steps in a pipeline, ms per step one after the other,
    H2D bytes, D2H bytes per step).

    Pipeline: two sets of device buffers (and a sequence for each) and three streams, so that the copies of steps
    i + 1 and i - 1 run beside the kernels of step i; every step still copies its own inputs in and its own
    outputs out inside the timed region, which starts before the first copy and ends after the last."""
    import torch
    from paper_2402_17764_b200 import binding as B
    x_host = stack.X_all.cpu().pin_memory()
    y_host = [torch.empty_like(stack.Y_all, device="cpu").pin_memory() for _ in range(2)]
    h2d, d2h = x_host.numel() * 2, y_host[0].numel() * 2

    # one after the other on one stream
    seq = B.Sequence(stack.layers)
    def step():
        stack.X_all.copy_(x_host, non_blocking=True)
        seq.forward()
        y_host[0].copy_(stack.Y_all, non_blocking=True)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    start, end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(steps):
        step()
    end.record()
    torch.cuda.synchronize()
    ms_serial = start.elapsed_time(end) / steps

    # the same steps as a pipeline
    X = [stack.X_all, torch.empty_like(stack.X_all)]
    Y = [stack.Y_all, torch.zeros_like(stack.Y_all)]
    second = []
    for packed, gamma, x, y, N in stack.layers:
        xo = (x.data_ptr() - stack.X_all.data_ptr()) // 2
        yo = (y.data_ptr() - stack.Y_all.data_ptr()) // 2
        second.append((packed, gamma, X[1][xo:xo + x.numel()].view_as(x), Y[1][yo:yo + y.numel()].view_as(y), N))
    seqs = [seq, B.Sequence(second)]
    s_in, s_run, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def run(n):
        copied_in = [None, None]   # per buffer set: events of its latest use
        computed = [None, None]
        copied_out = [None, None]
        first = last = None
        for i in range(n):
            b = i & 1
            with torch.cuda.stream(s_in):
                if i == 0:
                    first = torch.cuda.Event(enable_timing=True)
                    first.record()
                if computed[b] is not None:
                    s_in.wait_event(computed[b])        # the kernels of step i - 2 have read X[b]
                X[b].copy_(x_host, non_blocking=True)
                copied_in[b] = torch.cuda.Event()
                copied_in[b].record()
            with torch.cuda.stream(s_run):
                s_run.wait_event(copied_in[b])
                if copied_out[b] is not None:
                    s_run.wait_event(copied_out[b])     # the outputs of step i - 2 have left Y[b]
                seqs[b].forward(stream=s_run)
                computed[b] = torch.cuda.Event()
                computed[b].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(computed[b])
                y_host[b].copy_(Y[b], non_blocking=True)
                copied_out[b] = torch.cuda.Event()
                copied_out[b].record()
                if i == n - 1:
                    last = torch.cuda.Event(enable_timing=True)
                    last.record()
        torch.cuda.synchronize()
        return first.elapsed_time(last) / n

    run(max(warmup, 2))
    ms_pipe = run(steps)
    for sq in seqs:
        if B.poll_status(sq.workspace) != 0:
            raise RuntimeError("device status after the end-to-end steps")
    # both buffer sets received the same inputs: the same outputs must have come back
    if not torch.equal(y_host[0].view(torch.int16), y_host[1].view(torch.int16)):
        raise RuntimeError("the two buffer sets of the end-to-end pipeline disagree")
    for sq in seqs:
        sq.close()
    return ms_pipe, ms_serial, h2d, d2h


def time_forward_calls(fn, iters, warmup=3, repeats=1):
    """ms per call: `iters` calls between two events; with repeats > 1 the median of that many measurements."""
    import torch
    for _ in range(warmup):
        fn()
    out = []
    for _ in range(repeats):
        torch.cuda.synchronize()
        s, e = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        s.record()
        for _ in range(iters):
            fn()
        e.record()
        torch.cuda.synchronize()
        out.append(s.elapsed_time(e) / iters)
    return statistics.median(out)


def measure_int8_peak():
    """The int8 tensor ceiling of this GPU, measured now: (a) the library's tcgen05.mma kind::i8 issue loop (operands
    resident in shared memory, nothing but MMAs), (b) torch._int_mm on 8192^3 as library context.  TOP/s, 2 per MAC."""
    import torch
    from paper_2402_17764_b200 import binding as B
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    iters = 16384   # about 4.5 ms per launch
    ops = B.probe_int8_peak(iters, status)
    ms = time_forward_calls(lambda: B.probe_int8_peak(iters, status), 4, warmup=2, repeats=5)
    if int(status.item()) != 0:
        raise RuntimeError("the int8 probe's wait expired")
    out = {"issue_loop_TOPS": round(ops / ms / 1e9, 1), "issue_loop_ms": round(ms, 4),
           "issue_loop": "148 CTAs x 16384 x 4 tcgen05.mma kind::i8 128x256x32, random operand bytes, no loads in the loop"}
    try:
        a = torch.randint(-127, 128, (8192, 8192), dtype=torch.int8, device="cuda")
        b = torch.randint(-1, 2, (8192, 8192), dtype=torch.int8, device="cuda").t()
        ms_mm = time_forward_calls(lambda: torch._int_mm(a, b), 10, warmup=3, repeats=3)
        out["torch_int_mm_8192_TOPS"] = round(2.0 * 8192 ** 3 / ms_mm / 1e9, 1)
        del a, b
    except Exception as exc:  # library context only
        out["torch_int_mm_8192_TOPS"] = None
        out["torch_int_mm_error"] = str(exc)[:120]
    return out


def prefill_roofline(int8_peak):
    """The tensor-core GEMM alone (events around the matmul launch of a one-entry sequence) on the 13B-shaped up
    projection at 8192 tokens, against the int8 ceiling measured in this run."""
    import torch
    from paper_2402_17764_b200 import binding as B
    from paper_2402_17764_b200 import synthetic as S
    N, K, M = 13824, 5120, 8192
    st = Stack([S.LayerShape("up", N, K)], 1, M)
    seq = B.Sequence(st.layers)
    for _ in range(3):
        seq.forward()
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
    for a, b in pairs:
        seq.forward_stage(1)
        a.record()
        seq.forward_stage(2)
        b.record()
    torch.cuda.synchronize()
    assert B.poll_status(seq.workspace) == 0
    ms = statistics.median(a.elapsed_time(b) for a, b in pairs)
    ms_fwd = time_forward_calls(seq.forward, 10, warmup=2, repeats=3)
    seq.close()
    tops = st.int_ops / ms / 1e9
    peak = int8_peak["issue_loop_TOPS"]
    return {"bound": "tensor", "kernel": "prefill_gemm_kernel<2, true>", "workload": f"13b_prefill {N}x{K} M={M}",
            "achieved": round(tops, 1), "peak": peak,
            "peak_source": "measured in this run (tcgen05.mma kind::i8 issue loop)", "unit": "TOP/s",
            "frac": round(tops / peak, 4), "frac_of_nominal_4500": round(tops / 4500.0, 4), "traffic": None,
            "kernel_ms": round(ms, 4), "forward_ms_with_quantiser": round(ms_fwd, 4),
            "forward_TOPS_with_quantiser": round(st.int_ops / ms_fwd / 1e9, 1)}


def decode_block(stack, steps, warmup, peaks, barrier=None, e2e_steps=None):
    """roofline + e2e figures of one decode workload (one rank's view)."""
    t = time_sequence(stack, steps, warmup, barrier)
    ms_e2e, ms_e2e_serial, h2d, d2h = time_e2e(stack, e2e_steps or max(10, steps // 2), 3)
    return t, ms_e2e, ms_e2e_serial, h2d, d2h


def extras(peaks, int8_peak, weights70):
    """Other workloads of the benchmark definition, reported beside the headline (1 GPU only)."""
    import torch
    from paper_2402_17764_b200 import binding as B
    from paper_2402_17764_b200 import synthetic as S
    out = {}
    hbm = peaks["hbm_gbs"]
    tensor_peak = int8_peak["issue_loop_TOPS"]

    # single BitLinear, M=8, K=1536, N=4096 (fits L2: a latency number, not a bandwidth one)
    cfg = S.CONFIGS["single"]
    st = Stack(cfg["layers"], 1, 8, cfg["outlier_frac"], cfg["outlier_scale"])
    packed, gamma, X, Y, N = st.layers[0]
    ws = B.alloc_workspace(8, N, X.shape[1])
    us = time_forward_calls(lambda: B.forward(packed, gamma, X, N, Y=Y, workspace=ws), 200, repeats=3) * 1e3
    out["single_M8_K1536_N4096"] = {"us_per_call": round(us, 2), "note": "L2-resident, launch-bound"}
    del st

    # 7B-shaped batched decode: each shape as a sequence of distinct copies (> L2) so reads come from HBM
    cfg = S.CONFIGS["7b_batched"]
    res = {}
    for sh in cfg["layers"]:
        copies = max(2, int(400e6 // S.packed_weight_bytes(sh.N, sh.K)))
        w = Weights([sh], 1, copies=copies)
        for M in cfg["M"]:
            st = Stack([sh], 1, M, cfg["outlier_frac"], cfg["outlier_scale"], weights=w)
            t = time_sequence(st, 20, 3, min_timed_s=0.05)
            gbs = st.algorithmic_bytes / (t["ms"] * 1e-3) / 1e9
            tops = st.int_ops / (t["ms"] * 1e-3) / 1e12
            # which roof binds: streaming the packed weights once, or 2*M*N*K integer operations on the tensor cores
            t_hbm, t_tensor = st.algorithmic_bytes / (hbm * 1e9), st.int_ops / (tensor_peak * 1e12)
            res[f"{sh.N}x{sh.K}_M{M}"] = {"ms": round(t["ms"], 4), "ms_min": round(t["ms_min"], 4), "GB/s": round(gbs, 1),
                                          "frac_hbm_measured": round(gbs / hbm, 3), "TOPS": round(tops, 2),
                                          "frac_of_min_roof": round(max(t_hbm, t_tensor) / (t["ms"] * 1e-3), 3)}
            del st
        del w
    out["decode_7b_shapes"] = res

    # 13B-shaped prefill: bitlinear_forward (quantiser + tensor-core GEMM + epilogue)
    cfg = S.CONFIGS["13b_prefill"]
    res = {}
    for sh in cfg["layers"]:
        W = S.latent_weights(sh.N, sh.K, 0, device="cuda")
        packed, gamma = B.quantize_weights(W)
        del W
        for M in cfg["M"]:
            X = S.activations(M, sh.K, 0, device="cuda")
            Y = torch.empty((M, sh.N), dtype=torch.bfloat16, device="cuda")
            ws = B.alloc_workspace(M, sh.N, sh.K)
            iters = 20 if M <= 2048 else 8
            ms = time_forward_calls(lambda: B.forward(packed, gamma, X, sh.N, Y=Y, workspace=ws), iters, repeats=5)
            tops = 2.0 * M * sh.N * sh.K / (ms * 1e-3) / 1e12  # the whole forward: quantiser + GEMM + epilogue
            res[f"{sh.N}x{sh.K}_M{M}"] = {"ms": round(ms, 4), "TOPS": round(tops, 1),
                                          "frac_int8_nominal_4500": round(tops / 4500.0, 3),
                                          "frac_int8_measured_issue_loop": round(tops / tensor_peak, 3)}
            del X, Y, ws
    out["prefill_13b_shapes"] = res

    # RMSNorm fused into the activation quantiser (HBM-bound: 2 B read + 1 B written per element; inputs larger
    # than L2) next to the plain quantiser
    res = {}
    for M, K in [(16384, 8192), (32768, 5120)]:
        H = S.activations(M, K, 0, device="cuda")
        gain = torch.ones(K, dtype=torch.float32, device="cuda")
        Xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
        beta = torch.empty(M, dtype=torch.float32, device="cuda")
        rs = torch.empty(M, dtype=torch.int32, device="cuda")
        L = B.load_library()
        stream = torch.cuda.current_stream().cuda_stream
        ms_n = time_forward_calls(lambda: L.bitlinear_rmsnorm_quantize_acts(H.data_ptr(), gain.data_ptr(), 1e-5, M, K,
                                                                            Xq.data_ptr(), beta.data_ptr(), rs.data_ptr(), stream), 10, repeats=3)
        ms_p = time_forward_calls(lambda: L.bitlinear_quantize_acts(H.data_ptr(), M, K, Xq.data_ptr(), beta.data_ptr(),
                                                                    rs.data_ptr(), stream), 10, repeats=3)
        res[f"M{M}_K{K}"] = {"rmsnorm_quantiser_ms": round(ms_n, 4), "GB/s": round(3.0 * M * K / ms_n / 1e6, 1),
                             "frac_hbm_measured": round(3.0 * M * K / ms_n / 1e6 / hbm, 3),
                             "plain_quantiser_ms": round(ms_p, 4), "plain_GB/s": round(3.0 * M * K / ms_p / 1e6, 1)}
        del H, Xq
    out["rmsnorm_quantiser"] = res

    # SwiGLU fused into the activation quantiser of the down projection (2 x 2 B read + 1 B written per element; the
    # product silu(gate) * up is never written), at the feed-forward widths of the 7B- and 13B-shaped layers
    res = {}
    for M, K in [(8192, 11008), (8192, 13824)]:
        gate = S.activations(M, K, 0, device="cuda")
        up = S.activations(M, K, 1, device="cuda")
        Xq = torch.empty((M, K), dtype=torch.int8, device="cuda")
        beta = torch.empty(M, dtype=torch.float32, device="cuda")
        rs = torch.empty(M, dtype=torch.int32, device="cuda")
        L = B.load_library()
        stream = torch.cuda.current_stream().cuda_stream
        ms_s = time_forward_calls(lambda: L.bitlinear_swiglu_quantize_acts(gate.data_ptr(), up.data_ptr(), M, K, Xq.data_ptr(),
                                                                           beta.data_ptr(), rs.data_ptr(), stream), 10, repeats=3)
        res[f"M{M}_K{K}"] = {"swiglu_quantiser_ms": round(ms_s, 4), "GB/s": round(5.0 * M * K / ms_s / 1e6, 1),
                             "frac_hbm_measured": round(5.0 * M * K / ms_s / 1e6 / hbm, 3)}
        del gate, up, Xq
    out["swiglu_quantiser"] = res

    # the forward with 4-bit activations (Q_b = 7) beside the 8-bit one: the same kernels, another scale
    res = {}
    for (N, K, M) in [(11008, 4096, 1), (13824, 5120, 2048)]:
        W = S.latent_weights(N, K, 0, device="cuda")
        packed, gamma = B.quantize_weights(W)
        del W
        X = S.activations(M, K, 0, device="cuda")
        Y = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
        ws = B.alloc_workspace(M, N, K)
        ms4 = time_forward_calls(lambda: B.forward_act_bits(packed, gamma, X, N, 4, Y=Y, workspace=ws), 50)
        ms8 = time_forward_calls(lambda: B.forward(packed, gamma, X, N, Y=Y, workspace=ws), 50)
        res[f"{N}x{K}_M{M}"] = {"forward_4bit_ms": round(ms4, 4), "forward_8bit_ms": round(ms8, 4)}
        del X, Y, ws, packed
    out["act_bits_4"] = res

    # the 3B-shaped step with the RMSNorm fused into the quantiser of q, k, v, gate and up (130 of the 182 matrices)
    cfg = S.CONFIGS["3b_decode"]
    st = Stack(cfg["layers"], cfg["n_layers"], 1)
    shapes = list(cfg["layers"])
    gains = []
    for i in range(len(st.layers)):
        sh = shapes[i % len(shapes)]
        gains.append(torch.ones(sh.K, dtype=torch.float32, device="cuda") if sh.name in ("q", "k", "v", "gate", "up") else None)
    seq = B.Sequence(st.layers, gains=gains, norm_eps=1e-5)
    ms = time_forward_calls(seq.forward, 300, warmup=20, repeats=3)
    assert B.poll_status(seq.workspace) == 0
    out["3b_decode_step_with_rmsnorm"] = {"ms_per_step": round(ms, 4), "GB/s": round(st.algorithmic_bytes / ms / 1e6, 1),
                                          "normalised_matrices": sum(g is not None for g in gains)}
    seq.close()

    # the same step (without the RMSNorm) replayed from a CUDA graph that holds ten steps
    seq = B.Sequence(st.layers)
    seq.forward()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(10):
            seq.forward()
    ms = time_forward_calls(graph.replay, 30, warmup=3, repeats=3) / 10
    assert B.poll_status(seq.workspace) == 0
    out["3b_decode_step_cuda_graph"] = {"ms_per_step": round(ms, 4), "GB/s": round(st.algorithmic_bytes / ms / 1e6, 1),
                                        "steps_per_graph": 10}
    del graph
    seq.close()
    del st, seq

    # the 3B-shaped step on the base-3 format (five weights per byte: 4/5 of the bytes, a table look-up per stored byte)
    # beside the 2-bit step
    cfg = S.CONFIGS["3b_decode"]
    res = {}
    for trits in (False, True):
        st = Stack(cfg["layers"], cfg["n_layers"], 1, weights=Weights(cfg["layers"], cfg["n_layers"], trits=trits))
        t = time_sequence(st, 200, 20, min_timed_s=0.2)
        res["base3_1.6bit" if trits else "2bit"] = {
            "ms_per_step": round(t["ms"], 4), "ms_min": round(t["ms_min"], 4), "stored_bytes": st.weights.stored_bytes,
            "stored_GB/s": round(st.weights.stored_bytes / t["ms"] / 1e6, 1),
            "GB/s_of_2bit_bytes": round(st.algorithmic_bytes / t["ms"] / 1e6, 1)}
        del st
        torch.cuda.empty_cache()
    out["3b_decode_step_trits"] = res

    # 70B-shaped step at more tokens: 16 (the benchmark definition) and 176 (the batch size of the paper's throughput
    # comparison on the 70B model, Table 3; tensor-core GEMM).  Each against the roof that binds it: streaming the
    # packed weights once (HBM) or 2*M*N*K integer operations (tensor cores), whichever takes longer.
    cfg = S.CONFIGS["70b_decode"]
    res = {}
    for M in [16, 176]:
        st = Stack(cfg["layers"], cfg["n_layers"], M, weights=weights70)
        t = time_sequence(st, 5, 3, min_timed_s=0.2)
        ms = t["ms"]
        gbs = st.algorithmic_bytes / (ms * 1e-3) / 1e9
        tops = st.int_ops / (ms * 1e-3) / 1e12
        t_hbm, t_tensor = st.algorithmic_bytes / (hbm * 1e9), st.int_ops / (tensor_peak * 1e12)
        res[f"M{M}"] = {"ms_per_step": round(ms, 3), "ms_min": round(t["ms_min"], 3), "GB/s": round(gbs, 1),
                        "TOPS": round(tops, 1), "packed_bytes": st.algorithmic_bytes,
                        "roofline": {"bound": "hbm" if t_hbm >= t_tensor else "tensor",
                                     "hbm_time_ms": round(t_hbm * 1e3, 3), "tensor_time_ms": round(t_tensor * 1e3, 3),
                                     "frac": round(max(t_hbm, t_tensor) / (ms * 1e-3), 3),
                                     "peaks": f"HBM {hbm} GB/s (measured copy), int8 {tensor_peak} TOP/s (measured issue loop)"}}
        del st
        torch.cuda.empty_cache()
    out["decode_70b_step"] = res
    return out


# ---------------------------------------------------------------------------------------------------
# CPU oracle legs

def _bf16_bits(t):
    import numpy as np
    import torch
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


class OracleSample:
    """A bounded sample of a workload for the CPU oracle: a list of (N, K, M) matrices, each cut to at most `max_rows`
    output rows (the oracle's matmul is row by row, so the rate per weight does not depend on N)."""

    def __init__(self, matrices, what, max_rows=None):
        from oracle import load_oracle
        from paper_2402_17764_b200 import synthetic as S
        self.orc = load_oracle("timing")
        self.items = []
        self.bytes = 0
        self.int_ops = 0
        for i, (N, K, M) in enumerate(matrices):
            n = min(N, max_rows) if max_rows else N
            W = S.latent_weights(n, K, i)
            T, g = self.orc.quantize_weights(W.numpy())
            X = _bf16_bits(S.activations(M, K, i))
            self.items.append((T, g, X))
            self.bytes += S.packed_weight_bytes(n, K)
            self.int_ops += 2 * M * n * K
        # the oracle's loops are parallel over TOKENS: a sample of M tokens keeps at most M threads busy
        self.cores = min(self.orc.num_threads(), max(m for _, _, m in matrices))
        self.sample = what

    def step(self):
        for T, g, X in self.items:
            self.orc.forward(T, g, X)


def headline_sample():
    """70B-shaped step: the q and k projections of one layer (8192 x 8192 and 1024 x 8192) at M = 1."""
    return OracleSample([(8192, 8192, 1), (1024, 8192, 1)],
                        "2 of the 560 matrices of the 70B-shaped step (q 8192x8192, k 1024x8192, M=1): activation "
                        "quantiser + int32 matmul + dequantisation")


def time_oracle(smp, budget_s, threads=None):
    """-> (seconds per step, repetitions) within about budget_s of CPU time."""
    if threads:
        smp.orc.set_num_threads(threads)
    smp.step()
    t0 = time.perf_counter()
    smp.step()
    one = time.perf_counter() - t0
    reps = max(2, min(200, int(budget_s / max(one, 1e-4))))
    t0 = time.perf_counter()
    for _ in range(reps):
        smp.step()
    dt = (time.perf_counter() - t0) / reps
    if threads:
        smp.orc.set_num_threads(os.cpu_count() or 1)
    return dt, reps


def cpu_baseline(budget_s=8.0):
    """The oracle as it stands on the host cores: the headline workload's sample (all cores, and one thread), and the
    other workloads of the benchmark definition on bounded samples."""
    from paper_2402_17764_b200 import synthetic as S
    smp = headline_sample()
    dt, reps = time_oracle(smp, budget_s)
    out = {"value": round(smp.bytes / dt / 1e9, 3), "unit": UNIT, "cores": smp.cores, "kind": "oracle",
           "sample": f"{smp.sample}, {reps} repetitions"}
    dt1, reps1 = time_oracle(smp, 3.0, threads=1)
    out["one_thread"] = {"value": round(smp.bytes / dt1 / 1e9, 3), "unit": UNIT, "cores": 1, "repetitions": reps1}
    others = {}
    c1 = OracleSample([(4096, 1536, 8)], "config 1 in full: 4096x1536 at M=8")
    d, r = time_oracle(c1, 2.0)
    others["single_M8_K1536_N4096"] = {"value": round(c1.bytes / d / 1e9, 3), "unit": UNIT, "ms": round(d * 1e3, 3),
                                       "cores": c1.cores, "sample": f"{c1.sample}, {r} repetitions"}
    cfg = S.CONFIGS["3b_decode"]
    c2 = OracleSample([(sh.N, sh.K, 1) for sh in cfg["layers"]], "1 of 26 decoder layers of the 3B-shaped step (7 matrices, M=1)")
    d, r = time_oracle(c2, 4.0)
    others["3b_decode"] = {"value": round(c2.bytes / d / 1e9, 3), "unit": UNIT, "ms": round(d * 1e3, 3), "cores": c2.cores,
                           "sample": f"{c2.sample}, {r} repetitions"}
    for M in (1, 64):
        c3 = OracleSample([(sh.N, sh.K, M) for sh in S.CONFIGS["7b_batched"]["layers"]],
                          f"config 3: the three 7B shapes in full at M={M}", max_rows=None if M == 1 else 1024)
        d, r = time_oracle(c3, 2.0)
        others[f"7b_batched_M{M}"] = {"value": round(c3.bytes / d / 1e9, 3), "unit": UNIT, "TOPS": round(c3.int_ops / d / 1e12, 4),
                                      "ms": round(d * 1e3, 3), "cores": c3.cores,
                                      "sample": f"{c3.sample}{'' if M == 1 else ', first 1024 output rows of each'}, {r} repetitions"}
    c4 = OracleSample([(sh.N, sh.K, 512) for sh in S.CONFIGS["13b_prefill"]["layers"]],
                      "config 4 at M=512: both 13B shapes, first 256 output rows of each", max_rows=256)
    d, r = time_oracle(c4, 3.0)
    others["13b_prefill_M512"] = {"value": round(c4.int_ops / d / 1e12, 4), "unit": "TOP/s", "ms": round(d * 1e3, 3),
                                  "cores": c4.cores, "sample": f"{c4.sample}, {r} repetitions"}
    out["other_workloads"] = others
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    smp = headline_sample()
    for _ in range(args.warmup):
        smp.step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        smp.step()
    dt = time.perf_counter() - t0
    value = smp.bytes * args.steps / dt / 1e9
    line = {
        "impl": "reference", "metric": METRIC, "value": round(value, 3), "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": round(dt / args.steps * 1e3, 3),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "CPU oracle on the host cores; each step is a bounded sample"},
        "cpu_baseline": {"value": round(value, 3), "unit": UNIT, "cores": smp.cores, "kind": "oracle", "sample": smp.sample},
        "e2e": {"value": round(value, 3), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------------

def max_over_ranks(dist, values, device):
    """Replicas only: the one thing the ranks exchange is their device-side timings; the slowest rank counts."""
    if dist is None:
        return list(values)
    import torch
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def all_ranks_agree(dist, mine: bool, device) -> bool:
    """True only if every rank says so: the ranks repeat their timed rounds until ALL of them have measured enough, so
    that every rank enters the same barriers the same number of times."""
    if dist is None:
        return bool(mine)
    import torch
    flag = torch.tensor([1.0 if mine else 0.0], device=device)
    dist.all_reduce(flag, op=dist.ReduceOp.MIN)
    return bool(flag.item() > 0.5)


def aggregate_throughput(bytes_per_rank, n_ranks, ms):
    """Whole-job GB/s: every rank streams its own replica of the weights in `ms` (the maximum over ranks)."""
    return n_ranks * bytes_per_rank / (ms * 1e-3) / 1e9


def decode_roofline(bytes_per_launch, kernel_ms, peaks, ratio):
    achieved = bytes_per_launch / (kernel_ms * 1e-3) / 1e9
    return {"bound": "hbm", "kernel": "decode_mma_kernel<1>", "achieved": round(achieved, 1),
            "peak": peaks["hbm_gbs"], "peak_source": peaks["source"], "unit": "GB/s",
            "frac": round(achieved / peaks["hbm_gbs"], 4), "frac_of_nominal_8000": round(achieved / 8000.0, 4),
            "kernel_ms": round(kernel_ms, 4),
            "traffic": round(ratio * bytes_per_launch) if ratio else None}


def run_ours(args):
    import torch
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    else:
        torch.cuda.set_device(0)
    from paper_2402_17764_b200 import build, binding as B
    from paper_2402_17764_b200 import synthetic as S
    if rank == 0:
        build.build()
    if dist:
        dist.barrier()
    B.load_library()
    peaks = measured_peaks()
    ratio = ncu_traffic_ratio()

    cfg = S.CONFIGS[WORKLOAD]
    weights = Weights(cfg["layers"], cfg["n_layers"])
    stack = Stack(cfg["layers"], cfg["n_layers"], 1, weights=weights)
    barrier = (lambda: dist.barrier()) if dist else None

    sampler = ClockSampler(local)
    sampler.start()                      # before the warm-up: the timed rounds lie inside the sampled window
    t = time_sequence(stack, args.steps, args.warmup, barrier)
    clocks = sampler.stop()
    ms_e2e, ms_e2e_serial, h2d, d2h = time_e2e(stack, max(10, args.steps // 2), 3)

    ms_step, ms_min, ms_kernel, ms_e2e = max_over_ranks(dist, [t["ms"], t["ms_min"], t["kernel_ms"], ms_e2e], "cuda")
    n = world
    value = aggregate_throughput(stack.algorithmic_bytes, n, ms_step)
    e2e_value = aggregate_throughput(stack.algorithmic_bytes, n, ms_e2e)
    line = {
        "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": n, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": round(ms_step, 4), "ms_per_step_min": round(ms_min, 4),
        "rounds": t["rounds"], "timed_s": round(t["timed_s"], 3),
        "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": WORKLOAD, "M": 1, "matrices": len(stack.layers),
                   "packed_weight_bytes": stack.algorithmic_bytes,
                   "launch": "bitlinear_forward_sequence: quantiser launch + persistent matmul launch (programmatic "
                             "dependent, starts early) + small finishing launch per step",
                   "timing": f"rounds of {args.steps} steps until {MIN_TIMED_S} s are timed; ms_per_step is the median round",
                   "l2": "inputs (17.1 GB of weights per step) larger than L2; no flush needed",
                   "parallelism": "replicas only" if n > 1 else "1 GPU"},
        "roofline": decode_roofline(stack.algorithmic_bytes, ms_kernel, peaks, ratio),
        "e2e": {"value": round(e2e_value, 1), "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "ms_per_step": round(ms_e2e, 4),
                "how": "steps in a pipeline: two sets of device buffers, copy-in, kernels and copy-out on three streams; "
                       "every step copies its inputs from pinned host memory and its outputs back",
                "ms_per_step_one_after_the_other": round(ms_e2e_serial, 4)},
        "gpu_launches": 3 * args.steps * t["rounds"],
        "clocks": clocks,
    }
    if rank == 0 and n == 1:
        line["cpu_baseline"] = cpu_baseline()
        del stack
        torch.cuda.empty_cache()
        # the int8 tensor ceiling, measured now, and the prefill GEMM against it
        int8_peak = measure_int8_peak()
        line["int8_peak"] = int8_peak
        line["roofline_prefill"] = prefill_roofline(int8_peak)
        # the 3B-shaped step (805 MB per step: the fixed cost of a launch shows) with its own blocks
        cfg3 = S.CONFIGS["3b_decode"]
        st3 = Stack(cfg3["layers"], cfg3["n_layers"], 1)
        t3 = time_sequence(st3, 200, 20)
        e3, e3s, h3, d3 = time_e2e(st3, 200, 3)
        line["decode_3b_step"] = {
            "workload": "3b_decode", "matrices": len(st3.layers), "packed_weight_bytes": st3.algorithmic_bytes,
            "value": round(st3.algorithmic_bytes / t3["ms"] / 1e6, 1), "unit": UNIT, "ms_per_step": round(t3["ms"], 4),
            "ms_per_step_min": round(t3["ms_min"], 4), "rounds": t3["rounds"],
            "roofline": decode_roofline(st3.algorithmic_bytes, t3["kernel_ms"], peaks, ratio),
            "e2e": {"value": round(st3.algorithmic_bytes / e3 / 1e6, 1), "unit": UNIT, "h2d_bytes_per_step": h3,
                    "d2h_bytes_per_step": d3, "ms_per_step": round(e3, 4), "ms_per_step_one_after_the_other": round(e3s, 4)},
            "cpu_baseline": line["cpu_baseline"]["other_workloads"]["3b_decode"]}
        del st3
        torch.cuda.empty_cache()
        if not args.no_extras:
            line["extra"] = extras(peaks, int8_peak, weights)
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.barrier()
        dist.destroy_process_group()


def profile_case(name: str):
    """Small fixed cases for `ncu`: inputs larger than L2, well under a GB on the device, few launches."""
    import torch
    from paper_2402_17764_b200 import build, binding as B
    from paper_2402_17764_b200 import synthetic as S
    torch.cuda.set_device(0)
    build.build()
    if name.startswith("decode"):
        # 48 distinct 11008x4096 matrices (541 MB of packed weights) at M = 1; decode:M[:copies] overrides;
        # decode-trits[:M[:copies]]: the same matrices in the base-3 format (433 MB)
        parts = name.split(":")
        M = int(parts[1]) if len(parts) > 1 else 1
        copies = int(parts[2]) if len(parts) > 2 else 48
        trits = name.startswith("decode-trits")
        st = Stack([S.LayerShape("up", 11008, 4096)], 1, M, weights=Weights([S.LayerShape("up", 11008, 4096)], 1, copies=copies, trits=trits))
        seq = B.Sequence(st.layers, trits=trits)
        for _ in range(3):
            seq.forward()
        torch.cuda.synchronize()
        # every step runs both stages; the matmul launch is timed alone with events placed around it
        pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(20)]
        for a, b in pairs:
            seq.forward_stage(1)
            a.record()
            seq.forward_stage(2)
            b.record()
        torch.cuda.synchronize()
        assert B.poll_status(seq.workspace) == 0
        ms = sum(a.elapsed_time(b) for a, b in pairs) / len(pairs)
        print(json.dumps({"case": name, "packed_bytes_per_launch": st.weights.stored_bytes,
                          "matmul_kernel_ms": round(ms, 4), "GB/s": round(st.weights.stored_bytes / ms / 1e6, 1)}))
    elif name.startswith("prefill"):
        # 13824x5120 at M = 2048 (290 G integer operations per launch), or prefill:M, or prefill:M:N:K
        parts = name.split(":")
        M = int(parts[1]) if len(parts) > 1 else 2048
        N, K = (int(parts[2]), int(parts[3])) if len(parts) > 3 else (13824, 5120)
        W = S.latent_weights(N, K, 0, device="cuda")
        packed, gamma = B.quantize_weights(W)
        X = S.activations(M, K, 0, device="cuda")
        ws = B.alloc_workspace(M, N, K)
        for _ in range(3):
            B.forward(packed, gamma, X, N, workspace=ws)
        torch.cuda.synchronize()
        ms = time_forward_calls(lambda: B.forward(packed, gamma, X, N, workspace=ws), 20)
        ops = 2 * M * N * K
        print(json.dumps({"case": name, "int_ops_per_launch": ops, "forward_ms": round(ms, 4),
                          "TOPS": round(ops / ms / 1e9, 1)}))
    elif name.startswith("quantiser"):
        # activation quantiser alone on 16384 x 8192 bf16 (268 MB read, 134 MB written); quantiser:norm = with RMSNorm;
        # quantiser:swiglu = with SwiGLU on 8192 x 11008 gate and up inputs (361 MB read, 90 MB written)
        norm, swiglu = name.endswith(":norm"), name.endswith(":swiglu")
        M, K = (8192, 11008) if swiglu else (16384, 8192)
        H = S.activations(M, K, 0, device="cuda")
        gain = torch.ones(K, dtype=torch.float32, device="cuda")
        up = S.activations(M, K, 1, device="cuda") if swiglu else None
        fn = ((lambda: B.swiglu_quantize_acts(H, up)) if swiglu else
              (lambda: B.rmsnorm_quantize_acts(H, gain, 1e-5)) if norm else (lambda: B.quantize_acts(H)))
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ms = time_forward_calls(fn, 10)
        per_element = 5 if swiglu else 3
        print(json.dumps({"case": name, "bytes_per_launch": per_element * M * K, "ms": round(ms, 4),
                          "GB/s": round(float(per_element) * M * K / ms / 1e6, 1)}))
    elif name.startswith("peak"):
        # the int8 issue loop alone (iters x 4 MMAs per CTA; peak[:iters])
        iters = int(name.split(":")[1]) if ":" in name else 4096
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        ops = B.probe_int8_peak(iters, status)
        ms = time_forward_calls(lambda: B.probe_int8_peak(iters, status), 4, warmup=2, repeats=3)
        assert int(status.item()) == 0
        print(json.dumps({"case": name, "int_ops_per_launch": ops, "ms": round(ms, 4), "TOPS": round(ops / ms / 1e9, 1)}))
    else:
        raise SystemExit(f"unknown profile case {name}")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--profile-case", default=None, help="run a small fixed case (decode[:M[:copies]] | decode-trits[:M[:copies]] | prefill[:M[:N:K]] | quantiser[:norm|:swiglu] | peak[:iters]) and exit")
    args = ap.parse_args()
    if args.profile_case:
        profile_case(args.profile_case)
        return
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
