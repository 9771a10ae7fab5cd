#!/usr/bin/env python
"""Throughput of the quantized-linear hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config 4]

One *step* = one pass of the whole online path (rotation -> per-token quantization -> TLQ-decoding
tensor-core contraction -> epilogue) over every linear of the workload, through one `lrq_qlinear_stack` call.
The default workload is the largest one that fits a GPU: the video-DiT-shaped stack (28 blocks x 4 linears,
M = 32768 tokens, W4A8), inputs already in HBM; an L2 flush (a 512 MiB fill) runs between timed steps, outside
the timed events.  `value` is the whole-job TFLOP/s (2*M*N*K per linear, summed over ranks); `e2e` repeats the
measurement with the activations in pinned host memory and the outputs read back, copies inside the timed region.
`roofline` / `roofline_rotq` time the workload's dominant contraction and its largest rotate+quantize alone;
`per_config` carries the whole-step rate of the other four workloads and, for the FLUX-shaped one, the same two
objects plus the dense rotation's (the shapes the roofline targets name).

With --gpus N > 1 (under torchrun) every rank runs the same batch on its own GPU: tokens are independent,
the path has no exchange step, so ranks share nothing but the timing barrier ("weak" scaling).

--impl reference times the fp64 CPU oracle on the host cores on a bounded token sample of the same
workload and prints the same line with "impl": "reference".
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
sys.path.insert(0, ROOT)

from lrq_workloads import bf16_bits_to_f64, config_layers, default_clip_grid  # noqa: E402

# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) from the ncu captures summarised under
# profiles/, keyed by the kernel and layer the roofline object describes.  A key is dropped (traffic: null) when its
# kernel changes after the capture.
NCU_TRAFFIC_BYTES = {
    "qgemm cfg4 b0.fc1": 65.20e6 + 547.50e6,
    "qgemm cfg3 fc1": 27.10e6 + 169.40e6,
    "rotq cfg4 b0.fc2": 303.10e6 + 117.94e6,
    "rotq cfg3 fc2": 113.27e6 + 11.70e6,
    "rotgemm cfg3 qkv": 51.51e6 + 19.17e6 + 56.67e6 + 0.25e6,
}

# sm__pipe_tensor_cycles_active (% of elapsed cycles) of the same captures: the tensor pipe's own view of the
# contraction, beside the fraction of the measured matmul peak that `frac` reports
NCU_TENSOR_PIPE_PCT = {"qgemm cfg4 b0.fc1": 48.4, "qgemm cfg3 fc1": 54.2}

METRIC = "qlinear_tflops"
UNIT = "TFLOP/s"
ORACLE_SAMPLE_TOKENS = 128


def workload_name(cfg: int) -> str:
    return {0: "cfg0 single linear W3A4 M=256 K=N=1024",
            1: "cfg1 PixArt-shape block linears W4A8 M=4096 hidden=1152 (qkv, proj, fc1, fc2)",
            2: "cfg2 MMDiT-shape linears W3A4 M=4429 hidden=1536 G=128",
            3: "cfg3 FLUX-shape linears W4A4 M=4608 hidden=3072",
            4: "cfg4 video-DiT stack 28 blocks W4A8 M=32768 hidden=1152"}[cfg]


def config_dict(cfg: int, n_layers: int, out_dtype: str):
    """The `config` object of the JSON line: the same for both arms (the oracle arm computes in fp64 whatever the
    output type of the library)."""
    return {"workload": workload_name(cfg), "layers": n_layers, "out_dtype": out_dtype,
            "l2": "CUDA arm: flushed between timed steps (512 MiB fill outside the timed events)"}


def layer_flops(specs, M=None):
    return sum(2.0 * (s.M if M is None else M) * s.N * s.K for s in specs)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except Exception:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------ oracle arm
def oracle_step(orc, prepared):
    """One bounded-sample pass of the oracle over every layer; returns seconds."""
    t0 = time.perf_counter()
    for spec, T, X, R in prepared:
        orc.qlinear(X, T, spec.a_bits, spec.rot, spec.had_block, R)
    return time.perf_counter() - t0


def prepare_oracle(orc, specs, n_tok):
    g = default_clip_grid()
    out = []
    for s in specs:
        T = orc.tlq_quantize(s.weights().astype(np.float64), s.w_bits, s.group, 7, g, g)
        X = bf16_bits_to_f64(s.activations(n_tok))
        Rb = s.rotation_bf16()
        out.append((s, T, X, None if Rb is None else bf16_bits_to_f64(Rb)))
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle as orc
    orc.build()
    specs = config_layers(args.config)
    if args.config == 4:
        specs = specs[:4]          # one block of the stack is a bounded sample of 28 identical blocks
    n_tok = ORACLE_SAMPLE_TOKENS
    prepared = prepare_oracle(orc, specs, n_tok)
    for _ in range(max(1, min(args.warmup, 2))):
        oracle_step(orc, prepared)
    ts = [oracle_step(orc, prepared) for _ in range(args.steps)]
    sec = float(np.mean(ts))
    fl = layer_flops(specs, n_tok)
    val = fl / sec / 1e12
    sample = f"{n_tok} tokens of each linear (full K, N); work is linear in tokens"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": config_dict(args.config, len(config_layers(args.config)), args.out_dtype), "sample": sample,
            "tokens_per_s": n_tok / sec,
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------ ranks
def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (the per-step time of a multi-GPU run is the
    slowest rank's).  `dist` is torch.distributed with an initialised process group; works with gloo on CPU."""
    import torch
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


# ------------------------------------------------------------------------------------------ CUDA arm
class Workload:
    """One workload resident on the device: TLQ-quantized layers (quantized here, timed), activations, outputs, the
    argument arrays of its lrq_qlinear_stack call and a CUDA graph of that call."""

    def __init__(self, P, torch, cfg, dev, out_name, capture=True):
        self.P, self.torch, self.cfg, self.dev = P, torch, cfg, dev
        self.specs = config_layers(cfg)
        grid = default_clip_grid()
        self.ydt, y_torch = out_dtype(P, out_name)
        self.layers, self.Xs_host, self.Xs, self.Ys = [], [], [], []
        x_cache, y_cache = {}, {}
        self.tlq_ms, self.n_weights = 0.0, 0
        for s in self.specs:
            Wd = torch.from_numpy(s.weights()).to(dev)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            # 3-bit codes of a small batch are stored in their true packing (eight codes in three bytes): such a layer
            # is bound by streaming its weights once, and the small-tile contraction reads that layout
            layout = P.CODES_PACKED3 if (s.w_bits == 3 and s.M <= 512) else P.CODES_NIBBLE
            tl = P.lrq_tlq_quantize_weights(Wd, s.w_bits, s.group, 7, grid, grid, code_layout=layout)
            e1.record()
            torch.cuda.synchronize()
            self.tlq_ms += e0.elapsed_time(e1)
            self.n_weights += s.N * s.K
            R = None if s.rot != "dense" else bf16_tensor(torch, s.rotation_bf16()).to(dev)
            kind = P.ROT_DENSE if s.rot == "dense" else P.ROT_HADAMARD
            self.layers.append(P.QLayer(tl, s.N, s.K, kind, s.a_bits, s.had_block, R))
            key = (s.K, s.n_salient) if cfg == 4 else (s.seed,)
            if key not in x_cache:                       # the stack reuses one activation buffer per distinct K
                xh = bf16_tensor(torch, s.activations()).pin_memory()
                x_cache[key] = (xh, xh.to(dev))
            self.Xs_host.append(x_cache[key][0])
            self.Xs.append(x_cache[key][1])
            del Wd
        for s in self.specs:                              # outputs: one buffer per distinct N (reused across blocks)
            key = s.N if cfg == 4 else s.seed
            if key not in y_cache:
                y_cache[key] = torch.empty((s.M, s.N), dtype=y_torch, device=dev)
            self.Ys.append(y_cache[key])
        self.plan = P.StackPlan(self.layers, self.Xs, self.Ys, self.ydt)
        self.ws = torch.empty(self.plan.need, dtype=torch.uint8, device=dev)
        self.graph = None
        if capture:
            self.capture()

    def step_direct(self):
        self.P.lrq_qlinear_stack(self.plan, self.ws, self.torch.cuda.current_stream())

    def capture(self):
        # The step is captured once into a CUDA graph and replayed: the path is a fixed sequence of launches, and a
        # replay removes the host-side launch gaps between them (--no-graph times the plain stream-ordered calls).
        torch = self.torch
        stream = torch.cuda.current_stream()
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        with torch.cuda.stream(side):
            for _ in range(2):
                self.step_direct()       # first-call set-up (function attributes, occupancy queries) happens outside the capture
        stream.wait_stream(side)
        torch.cuda.synchronize()
        self.graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self.graph):
            self.step_direct()

    def step(self):
        if self.graph is not None:
            self.graph.replay()
        else:
            self.step_direct()

    def flops(self):
        return layer_flops(self.specs)

    def launches_per_step(self):
        # kernels of this library per step: rotate+quantize and contraction per layer, one more (the rotation GEMM
        # before its quantizer) per dense layer; the two memsets of a dense rotation are not kernels
        return 2 * len(self.specs) + sum(1 for s in self.specs if s.rot == "dense")

    def close(self):
        for L in self.layers:
            L.close()


def bf16_tensor(torch, bits):
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)


def kernel_objects(P, torch, W, timed, peaks, out_name, gemm_impl=0, want_dense=False):
    """Roofline objects of one workload's kernels, each timed alone (L2 flushed between launches): the contraction
    with the most flops (tensor bound), the Hadamard rotate+quantize with the most bytes (HBM bound) and, on request,
    the dense rotation with the most flops (tensor bound; rotation GEMM + its quantizer pass)."""
    specs, layers, stream = W.specs, W.layers, torch.cuda.current_stream()
    cfg = W.cfg
    out = {}
    # "timed alone": the steps that ran before leave the part at the clock its power cap allows; two idle seconds
    # let it return to the state in which the burst peaks these kernels are compared with were measured
    torch.cuda.synchronize()
    time.sleep(2.0)
    big = max(range(len(specs)), key=lambda i: specs[i].N * specs[i].K * specs[i].M)
    s, L = specs[big], layers[big]
    q, sc, zp = P.lrq_rotate_quantize_act(W.Xs[big], L.kind, s.a_bits, s.had_block, L.R)
    impl = 2 if L.tlq.code_layout == P.CODES_PACKED3 else gemm_impl
    gq = torch.cuda.CUDAGraph()                       # one launch per replay: no host call inside the timed events
    P.lrq_qgemm_codes(L, q, sc, zp, W.ydt, impl, W.Ys[big], stream)
    torch.cuda.synchronize()
    with torch.cuda.graph(gq):
        P.lrq_qgemm_codes(L, q, sc, zp, W.ydt, impl, W.Ys[big])
    gemm_ms = float(np.mean(timed(gq.replay, 20)))
    gemm_tf = 2.0 * s.M * s.N * s.K / (gemm_ms * 1e-3) / 1e12
    if L.tlq.code_layout == P.CODES_PACKED3:
        # a small batch: every byte is moved once and the tensor cores idle; algorithmic bytes = activation codes +
        # 3-bit weight codes + level tables + per-token / per-channel terms + outputs
        G = s.group if s.group > 0 else s.K
        esz = 4 if out_name == "f32" else 2
        nbytes = s.M * s.K * s.a_bits / 8.0 + s.N * s.K * 3 / 8.0 + s.N * (s.K // G) * 8 * 4.0 + 8.0 * s.M + 4.0 * s.N + s.M * s.N * esz
        gbs = nbytes / (gemm_ms * 1e-3) / 1e9
        out["roofline"] = {"kernel": f"qgemm (small-tile, packed 3-bit codes) cfg{cfg} {s.name} {s.M}x{s.N}x{s.K} W3A{s.a_bits} out {out_name}",
                           "bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                           "traffic": None, "algorithmic_bytes": nbytes, "tflops": gemm_tf,
                           "peak_source": peaks["source"] + " copy bandwidth; a launch of a few microseconds is latency-bound, not bandwidth-bound",
                           "ms": gemm_ms}
    else:
        out["roofline"] = {"kernel": f"qgemm cfg{cfg} {s.name} {s.M}x{s.N}x{s.K} W{s.w_bits}A{s.a_bits} out {out_name}", "bound": "tensor",
                           "achieved": gemm_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": gemm_tf / peaks["bf16_tflops"],
                           "traffic": NCU_TRAFFIC_BYTES.get(f"qgemm cfg{cfg} {s.name}") if out_name == "f32" else None,
                           "traffic_unit": "bytes per launch (ncu dram read + write)", "algorithmic_flops": 2.0 * s.M * s.N * s.K,
                           "tensor_pipe_active_pct_ncu": NCU_TENSOR_PIPE_PCT.get(f"qgemm cfg{cfg} {s.name}") if out_name == "f32" else None,
                           "peak_source": peaks["source"] + " burst bf16 (kernel timed alone)", "ms": gemm_ms}
    del q, sc, zp
    had = [i for i in range(len(specs)) if specs[i].rot == "hadamard"]
    if had:
        kbig = max(had, key=lambda i: specs[i].K * specs[i].M)
        sr, Lr = specs[kbig], layers[kbig]
        rq = P.lrq_rotate_quantize_act(W.Xs[kbig], Lr.kind, sr.a_bits, sr.had_block, Lr.R)
        rot_ms = float(np.mean(timed(lambda: P.lrq_rotate_quantize_act(W.Xs[kbig], Lr.kind, sr.a_bits, sr.had_block, Lr.R,
                                                                       stream=stream, out=rq), 20)))
        rot_bytes = sr.M * (2.0 * sr.K + sr.K * sr.a_bits / 8.0 + 8.0)
        rot_gbs = rot_bytes / (rot_ms * 1e-3) / 1e9
        out["roofline_rotq"] = {"kernel": f"rotq cfg{cfg} {sr.name} {sr.M}x{sr.K} B{sr.had_block} A{sr.a_bits}", "bound": "hbm",
                                "achieved": rot_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": rot_gbs / peaks["hbm_gbs"],
                                "traffic": NCU_TRAFFIC_BYTES.get(f"rotq cfg{cfg} {sr.name}"),
                                "peak_source": peaks["source"] + " copy bandwidth", "ms": rot_ms, "algorithmic_bytes": rot_bytes}
        del rq
    dense = [i for i in range(len(specs)) if specs[i].rot == "dense"]
    if want_dense and dense:
        d = max(dense, key=lambda i: specs[i].K * specs[i].K * specs[i].M)
        sd, Ld = specs[d], layers[d]
        need = Ld.workspace_bytes(sd.M)
        wsd = torch.empty(need, dtype=torch.uint8, device=W.dev)
        rq = P.lrq_rotate_quantize_act(W.Xs[d], Ld.kind, sd.a_bits, 0, Ld.R, workspace=wsd)
        d_ms = float(np.mean(timed(lambda: P.lrq_rotate_quantize_act(W.Xs[d], Ld.kind, sd.a_bits, 0, Ld.R, workspace=wsd,
                                                                     stream=stream, out=rq), 20)))
        d_tf = 2.0 * sd.M * sd.K * sd.K / (d_ms * 1e-3) / 1e12
        out["roofline_rotdense"] = {"kernel": f"rotgemm+quantizer cfg{cfg} {sd.name} {sd.M}x{sd.K}x{sd.K} A{sd.a_bits}", "bound": "tensor",
                                    "achieved": d_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                                    "frac": d_tf / peaks["bf16_tflops"], "traffic": NCU_TRAFFIC_BYTES.get(f"rotgemm cfg{cfg} {sd.name}"),
                                    "algorithmic_flops": 2.0 * sd.M * sd.K * sd.K,
                                    "peak_source": peaks["source"] + " burst bf16 (both kernels of the dense path timed together)",
                                    "ms": d_ms}
        del rq, wsd
        if sd.K % 128 == 0:
            # the same layer with its rotation kept in the factors of the dual transformation (seeded block rotations
            # around a staggered reordering): rotate+quantize of all tokens, beside the dense-matrix path above
            Bd, R1, perm, R2 = sd.dual_factors()
            dual = P.DualRotation(Bd, bf16_tensor(torch, R1).to(W.dev), torch.from_numpy(perm).to(W.dev),
                                  bf16_tensor(torch, R2).to(W.dev))
            wsu = torch.empty(10 * sd.M * sd.K + 4096, dtype=torch.uint8, device=W.dev)
            rq = P.lrq_rotate_quantize_act(W.Xs[d], P.ROT_DUAL, sd.a_bits, dual=dual, workspace=wsu)
            u_ms = float(np.mean(timed(lambda: P.lrq_rotate_quantize_act(W.Xs[d], P.ROT_DUAL, sd.a_bits, dual=dual, workspace=wsu,
                                                                         stream=stream, out=rq), 20)))
            out["rotdual"] = {"kernel": f"dual rotation (two block-diagonal products, reordering between) + quantizer cfg{cfg} {sd.name} "
                                        f"{sd.M}x{sd.K} Bd{Bd} A{sd.a_bits}", "ms": u_ms, "dense_path_ms": d_ms,
                              "algorithmic_flops": 2.0 * sd.M * sd.K * Bd * 4}
            del rq, wsu, dual
    return out


def run_cuda(args):
    import torch
    import torch.distributed as dist
    import paper_2508_03485_b200 as P

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    P.load_library()

    W = Workload(P, torch, args.config, dev, args.out_dtype, capture=not args.no_graph)
    specs, layers, Xs, Ys, Xs_host, ydt = W.specs, W.layers, W.Xs, W.Ys, W.Xs_host, W.ydt
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def timed(fn, n, flush_between=True):
        evs = []
        for _ in range(n):
            if flush_between:
                flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            evs.append((a, b))
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warm = max(3, args.warmup)
    for _ in range(warm):
        flush.fill_(1); W.step()
    barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    ms = timed(W.step, args.steps)
    barrier()
    ms_step = float(np.mean(ms))

    # ---- end to end: pinned host activations in, outputs back to pinned host memory, copies timed
    uniq_x = {id(h): (h, d) for h, d in zip(Xs_host, Xs)}
    uniq_y = {id(y): y for y in Ys}
    y_host = {k: torch.empty(y.shape, dtype=y.dtype).pin_memory() for k, y in uniq_y.items()}
    h2d = sum(h.numel() * 2 for h, _ in uniq_x.values())
    d2h = sum(y.numel() * y.element_size() for y in uniq_y.values())

    # One lrq_qlinear call per layer (and token chunk) on the compute stream; uploads run on a second stream and
    # read-backs on a third.  An output buffer is read back after its last writer.
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    first_reader, last_writer = {}, {}
    for i, (x, y) in enumerate(zip(Xs, Ys)):
        first_reader.setdefault(id(x), i)
        last_writer[id(y)] = i

    # A large batch goes through in token chunks (tokens are independent through the whole path): chunk c's outputs
    # travel back to the host while chunk c + 1 is computed, and its activations arrive while chunk c - 1 is computed.
    # The first and the last chunk are small: the kernels wait for the first chunk's upload only, and only the last
    # chunk's read-back is left over when they are done.
    m_all = Xs[0].shape[0]
    chunked = m_all >= 16384 and m_all % 16 == 0 and all(x.shape[0] == m_all for x in Xs)
    bounds = [m_all * f // 16 for f in (0, 2, 7, 12, 15, 16)] if chunked else [0, m_all]
    nch = len(bounds) - 1

    def e2e_step():
        s_in.wait_stream(stream)          # the previous step's kernels have read the activation buffers
        for c in range(nch):
            rows = slice(bounds[c], bounds[c + 1])
            with torch.cuda.stream(s_in):
                for h, d in uniq_x.values():
                    d[rows].copy_(h[rows], non_blocking=True)
                uploaded = torch.cuda.Event()
                uploaded.record(s_in)
            stream.wait_event(uploaded)
            for i, (L, x, y) in enumerate(zip(layers, Xs, Ys)):
                P.lrq_qlinear(L, x[rows], ydt, out=y[rows], workspace=W.ws, stream=stream)
                if last_writer[id(y)] == i:
                    done = torch.cuda.Event()
                    done.record(stream)
                    s_out.wait_event(done)
                    with torch.cuda.stream(s_out):
                        y_host[id(y)][rows].copy_(y[rows], non_blocking=True)
        stream.wait_stream(s_out)

    for _ in range(2):
        e2e_step()
    barrier()
    e2e_ms = float(np.mean(timed(e2e_step, max(2, min(args.steps, 10)))))
    barrier()
    clocks = sampler.stop() if rank == 0 else None

    if world > 1:
        ms_step, e2e_ms = max_over_ranks([ms_step, e2e_ms], dist, dev)

    flops = W.flops()
    tokens = sum(s.M for s in specs) / len(specs) if args.config != 4 else specs[0].M
    value = world * flops / (ms_step * 1e-3) / 1e12
    e2e_val = world * flops / (e2e_ms * 1e-3) / 1e12

    line = None
    if rank == 0:
        peaks = measured_peaks()
        # ---- per-kernel roofline objects of this workload, measured live
        objs = kernel_objects(P, torch, W, timed, peaks, args.out_dtype, args.gemm_impl, want_dense=True)
        extra = {}
        if not args.quick:
            # the same step and its dominant contraction with 16-bit outputs (the paper runs FP16 inference; the fp32
            # output stream of the largest layer is 1.5 TB/s)
            if args.out_dtype == "f32":
                W16 = Workload(P, torch, args.config, dev, "f16", capture=not args.no_graph)
                for _ in range(3):
                    flush.fill_(1); W16.step()
                ms16 = float(np.mean(timed(W16.step, max(3, min(args.steps, 10)))))
                o16 = kernel_objects(P, torch, W16, timed, peaks, "f16", args.gemm_impl)["roofline"]
                extra["out_f16"] = {"ms_per_step": ms16, "value": flops / (ms16 * 1e-3) / 1e12, "unit": UNIT,
                                    "roofline": {k: o16[k] for k in ("kernel", "achieved", "peak", "frac", "ms")}}
                W16.close(); del W16
                torch.cuda.empty_cache()
            # ---- the other workloads: whole-step rate, and for the FLUX-shaped one the kernels the roofline targets name
            per = []
            for c in [c for c in (3, 2, 1, 0) if c != args.config]:
                Wc = Workload(P, torch, c, dev, args.out_dtype, capture=not args.no_graph)
                for _ in range(3):
                    flush.fill_(1); Wc.step()
                msc = float(np.mean(timed(Wc.step, 10)))
                ent = {"config": c, "workload": workload_name(c), "layers": len(Wc.specs), "ms_per_step": msc,
                       "value": Wc.flops() / (msc * 1e-3) / 1e12, "unit": UNIT,
                       "tokens_per_s": (sum(s_.M for s_ in Wc.specs) / len(Wc.specs)) / (msc * 1e-3)}
                if c in (3, 0):
                    ent.update(kernel_objects(P, torch, Wc, timed, peaks, args.out_dtype, args.gemm_impl, want_dense=True))
                per.append(ent)
                Wc.close(); del Wc
                torch.cuda.empty_cache()
            extra["per_config"] = per
        # ---- CPU baseline: the oracle, as it stands, on a bounded token sample
        import oracle as orc
        orc.build()
        osp = specs[:4]
        prepared = prepare_oracle(orc, osp, ORACLE_SAMPLE_TOKENS)
        oracle_step(orc, prepared)
        osec = float(np.mean([oracle_step(orc, prepared) for _ in range(3)]))
        cpu_val = layer_flops(osp, ORACLE_SAMPLE_TOKENS) / osec / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": config_dict(args.config, len(specs), args.out_dtype),
            "run": {"launch": "one CUDA graph replay of lrq_qlinear_stack per step" if W.graph is not None else "stream-ordered launches",
                    "parallelism": f"replicated batch x{world}, no collective",
                    "whole_step_peak_note": "a whole step runs for tens of milliseconds under the power cap: compare it with "
                                            f"the sustained bf16 figure ({peaks['bf16_tflops_sustained']:.0f} TFLOP/s); kernels "
                                            "timed alone are compared with the burst figure"},
            "tokens_per_s": world * tokens / (ms_step * 1e-3),
            "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": e2e_ms, "launch": f"one lrq_qlinear call per layer and token chunk ({nch} chunk(s)); copies on two side streams"},
            "gpu_launches": args.steps * W.launches_per_step(),
            "clocks": clocks, "roofline": objs["roofline"], "roofline_rotq": objs.get("roofline_rotq"),
            "cpu_baseline": {"value": cpu_val, "unit": UNIT, "cores": orc.num_threads(), "kind": "oracle",
                             "sample": f"{ORACLE_SAMPLE_TOKENS} tokens of each of the first {len(osp)} linears (full K, N)",
                             "tokens_per_s": ORACLE_SAMPLE_TOKENS / osec},
            "tlq_weight_quantization": {"weights_per_s": W.n_weights / (W.tlq_ms * 1e-3), "ms": W.tlq_ms},
        }
        for k in ("roofline_rotdense", "rotdual"):
            if k in objs:
                line[k] = objs[k]
        line.update(extra)
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return line


def run_kernel(args):
    """Micro-benchmark of one kernel on one layer of the chosen workload (also the command the ncu captures
    under profiles/ use): --kernel rotq | qgemm | tlq, --layer index, --tokens M override."""
    import torch
    import paper_2508_03485_b200 as P
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    s = config_layers(args.config)[args.layer]
    M = args.tokens or s.M
    grid = default_clip_grid()
    stream = torch.cuda.current_stream()
    Wd = torch.from_numpy(s.weights()).to(dev)
    # as in the whole-step workload: 3-bit codes of a small batch are stored packed and take the small-tile kernel
    packed = s.w_bits == 3 and M <= 512
    tl = P.lrq_tlq_quantize_weights(Wd, s.w_bits, s.group, 7, grid, grid,
                                    code_layout=P.CODES_PACKED3 if packed else P.CODES_NIBBLE)
    if packed:
        args.gemm_impl = 2
    R = None if s.rot != "dense" else torch.from_numpy(s.rotation_bf16().view(np.int16)).view(torch.bfloat16).to(dev)
    kind = P.ROT_DENSE if s.rot == "dense" else P.ROT_HADAMARD
    L = P.QLayer(tl, s.N, s.K, kind, s.a_bits, s.had_block, R)
    X = torch.from_numpy(s.activations(min(M, 4096)).view(np.int16)).view(torch.bfloat16).to(dev)
    if M > X.shape[0]:
        X = X.repeat((M + X.shape[0] - 1) // X.shape[0], 1)[:M].contiguous()
    rq = P.lrq_rotate_quantize_act(X, kind, s.a_bits, s.had_block, R)
    ydt, y_torch = out_dtype(P, args.out_dtype)
    Y = torch.empty((M, s.N), dtype=y_torch, device=dev)
    ws = torch.empty(max(256, L.workspace_bytes(M)), dtype=torch.uint8, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    if args.kernel == "rotq":
        fn = lambda: P.lrq_rotate_quantize_act(X, kind, s.a_bits, s.had_block, R, workspace=ws, stream=stream, out=rq)
        units, unit = M * (2.0 * s.K + s.K * s.a_bits / 8.0 + 8.0) / 1e9, "GB/s"
    elif args.kernel == "qgemm":
        fn = lambda: P.lrq_qgemm_codes(L, rq[0], rq[1], rq[2], ydt, args.gemm_impl, Y, stream)
        units, unit = 2.0 * M * s.N * s.K / 1e12, "TFLOP/s"
    elif args.kernel == "ars":
        fn = lambda: P.lrq_ars_select(X, 1.0, stream)
        units, unit = M * 2.0 * s.K / 1e9, "GB/s"
    else:
        fn = lambda: P.lrq_tlq_quantize_weights(Wd, s.w_bits, s.group, 7, grid, grid)
        units, unit = s.N * s.K / 1e9, "Gweights/s"
    for _ in range(max(1, args.warmup)):
        fn()
    torch.cuda.synchronize()
    if not args.no_graph and args.kernel in ("rotq", "qgemm"):
        call = fn
        if args.kernel == "rotq":
            call = lambda: P.lrq_rotate_quantize_act(X, kind, s.a_bits, s.had_block, R, workspace=ws, out=rq)
        elif args.kernel == "qgemm":
            call = lambda: P.lrq_qgemm_codes(L, rq[0], rq[1], rq[2], ydt, args.gemm_impl, Y)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            call()
        fn = g.replay
    ts = []
    for _ in range(args.steps):
        flush.fill_(1)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream); fn(); b.record(stream)
        ts.append((a, b))
    torch.cuda.synchronize()
    ms = [a.elapsed_time(b) for a, b in ts]
    print(json.dumps({"kernel": args.kernel, "layer": s.name, "M": M, "K": s.K, "N": s.N, "rot": s.rot,
                      "had_block": s.had_block, "w_bits": s.w_bits, "a_bits": s.a_bits, "out_dtype": args.out_dtype,
                      "ms_mean": float(np.mean(ms)), "ms_min": float(np.min(ms)),
                      "rate_mean": units / (float(np.mean(ms)) * 1e-3), "rate_best": units / (float(np.min(ms)) * 1e-3),
                      "unit": unit, "status": P.lrq_device_status()}))


def out_dtype(P, name):
    import torch
    return {"f32": (P.F32, torch.float32), "f16": (P.F16, torch.float16), "bf16": (P.BF16, torch.bfloat16)}[name]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--config", type=int, default=4, choices=[0, 1, 2, 3, 4])
    ap.add_argument("--quick", action="store_true", help="only the chosen workload: no 16-bit-output leg, no per_config list")
    ap.add_argument("--gemm-impl", type=int, default=0, choices=[0, 1, 2],
                    help="kernel timed alone for the roofline object: 0 large-tile tcgen05, 1 CUDA-core baseline, 2 small-tile tcgen05")
    ap.add_argument("--no-graph", action="store_true", help="time plain launches instead of a CUDA graph replay of the step")
    ap.add_argument("--kernel", default=None, choices=["rotq", "qgemm", "tlq", "ars"], help="time one kernel only")
    ap.add_argument("--layer", type=int, default=0, help="layer index of the workload for --kernel")
    ap.add_argument("--out-dtype", default="f32", choices=["f32", "f16", "bf16"], help="type of the layer outputs Y")
    ap.add_argument("--tokens", type=int, default=0, help="override M for --kernel")
    args = ap.parse_args()
    if args.kernel:
        run_kernel(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
