#!/usr/bin/env python
"""Benchmark of libmipgemm on B200: one JSON line per run.

A *step* is one pass of the hot path over one batch of synthetic input: every GEMM (or
convolution) of a workload, launched back to back on one stream through the C ABI and
replayed as one CUDA graph.  The headline workload is the square s8*s8->s32 sweep
M=N=K in {1024 .. 16384}; the default run also times every other configuration of the
benchmark definition (512^3, the misaligned 1000x3001x777 accumulate case, the 53
ResNet-50 v1.5 convolutions at batch 32 and 128, the 21 BERT encoder GEMMs, the 16 decode
GEMMs with and without the constant-weights promise) and reports them under "workloads",
each with its roofline fractions, the clocks sampled during its timed region, the host-side
cost of a call and a sampled comparison of the very buffers that were timed with the CPU
oracle.

    python bench.py [--gpus N] [--steps K] [--warmup W]
                    [--workload all|square|gemm512|ragged|bert|resnet|skinny|paper_b1|attention|layouts]
    python bench.py --impl reference ...      # the CPU oracle, timed on the host cores

Under torchrun (N > 1) every rank runs the same per-GPU workload on its own device
(independent problems, no data-path collective: weak scaling); the time is the maximum
over ranks and the value is the aggregate over all ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2506_11728_b200 import inputs, sharding  # noqa: E402  (bytes / bookkeeping only, no arithmetic)

NOMINAL_INT8_TOPS = 4500.0
NOMINAL_BF16_TFLOPS = 2250.0
NOMINAL_HBM_GBS = 8000.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes (read + written) per launch of each workload's dominant kernel, taken from ncu captures
TRAFFIC_FILE = os.path.join(ROOT, "bench_ncu_traffic.json")


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        d["_source"] = "measured"
        return d
    d = dict(FALLBACK_PEAKS)
    d["_source"] = "fallback"
    return d


def load_traffic(name):
    try:
        with open(TRAFFIC_FILE) as f:
            return json.load(f).get(name, {}).get("dram_bytes_per_launch")
    except (OSError, ValueError):
        return None


def rnd(x, digits=4):
    """Shortens a float for the JSON line (significant digits, not decimals)."""
    if x is None or isinstance(x, (int, str, bool)):
        return x
    if x == 0 or not np.isfinite(x):
        return x
    return float("%.*g" % (digits, x))


# --------------------------------------------------------------------------- workloads
class Problem:
    """One library call: shapes, algorithmic ops/bytes, the device buffers it runs on and the host
    copies of its operands (kept for the oracle comparison)."""

    def __init__(self, name, kind, ops, nbytes):
        self.name, self.kind, self.ops, self.bytes = name, kind, float(ops), float(nbytes)
        self.calls = []          # zero-argument callables (one per rotation slot)
        self.count = 1           # launches per step when there is one call (layer multiplicity)
        self.host = None         # host-side operands
        self.accumulate = False
        self.mode = "s8"
        self.out_bytes = 0.0     # bytes of C written per launch (write-rate view)


class Workload:
    def __init__(self, name, probs, unit, metric, text, bound, kernel, l2_note):
        self.name, self.probs, self.unit, self.metric, self.text = name, probs, unit, metric, text
        self.bound, self.kernel, self.l2_note = bound, kernel, l2_note
        self.groups = []
        for p in probs:
            self.groups.append((p, p.count if len(p.calls) == 1 else len(p.calls)))
        self.launches_per_step = sum(r for (_p, r) in self.groups)
        self.step_ops = sum(p.ops * r for (p, r) in self.groups)
        self.step_bytes = sum(p.bytes * r for (p, r) in self.groups)
        self.step_out_bytes = sum(p.out_bytes * r for (p, r) in self.groups)
        self.steps_run = 0       # how often every problem has been launched (accumulating problems need it)


def _dev_bytes(torch, arr):
    return torch.from_numpy(arr.view(np.uint8)).cuda(non_blocking=False)


def _gemm_problem(torch, mg, name, M, N, K, A, B, mode="s8", lda=None, ldb=None, ldc=None, C0=None, sets=1):
    """One GEMM call.  ``sets`` > 1: that many copies of the operands and of C, used in turn, so that a
    small problem does not simply sit in the L2 (copy r holds A and B with their rows rotated by r: a
    device-side copy; the oracle comparison rotates the host arrays the same way)."""
    lda, ldb, ldc = lda or K, ldb or K, ldc or N
    acc = C0 is not None
    fn = mg.mipgemm_s8s8s32 if mode == "s8" else mg.mipgemm_u8s8s32
    p = Problem(name, "gemm", 2.0 * M * N * K, M * K + N * K + (8.0 if acc else 4.0) * M * N)
    dA0, dB0 = _dev_bytes(torch, A), _dev_bytes(torch, B)
    for r in range(sets):
        dA = dA0 if r == 0 else torch.roll(dA0.view(M, lda), r, 0).reshape(-1).contiguous()
        dB = dB0 if r == 0 else torch.roll(dB0.view(N, ldb), r, 0).reshape(-1).contiguous()
        dC = _dev_bytes(torch, C0).view(torch.int32) if acc else torch.empty(M * ldc, dtype=torch.int32, device="cuda")
        p.calls.append(lambda dA=dA, dB=dB, dC=dC: fn(M, N, K, dA, lda, dB, ldb, dC, ldc, 1 if acc else 0))
        p.bufs = (dA, dB, dC)        # the last copy: the one the oracle comparison reads
    p.dims, p.ld, p.host, p.accumulate, p.mode, p.sets = (M, N, K), (lda, ldb, ldc), (A, B, C0), acc, mode, sets
    p.out_bytes = 4.0 * M * N
    return p


def build_square(torch, mg, sizes):
    probs = []
    for n in sizes:
        A = inputs.uniform_s8(n * n, inputs.seed_for(2, n) + 1)
        B = inputs.uniform_s8(n * n, inputs.seed_for(2, n) + 2)
        probs.append(_gemm_problem(torch, mg, "square_%d" % n, n, n, n, A, B))
    return Workload("square", probs, "TOPS", "int8_gemm_tops",
                    "square s8*s8->s32 sweep M=N=K in %s, uniform int8, accumulate=0" % sizes, "tensor",
                    "mip_dense_kernel", "operands + outputs of one step exceed the 126 MB L2 many times over")


def build_gemm512(torch, mg):
    n = 512
    A = inputs.uniform_s8(n * n, inputs.seed_for(1, 1))
    B = inputs.uniform_s8(n * n, inputs.seed_for(1, 2))
    return Workload("gemm512", [_gemm_problem(torch, mg, "gemm_512", n, n, n, A, B, sets=160)], "TOPS",
                    "int8_gemm_tops", "single GEMM s8*s8->s32 M=N=K=512, uniform int8, accumulate=0", "tensor",
                    "mip_dense_kernel", "160 copies of the 1.6 MB problem used in turn (250 MB > L2); a launch-latency "
                    "measurement at this size")


def build_ragged(torch, mg):
    M, N, K = 1000, 3001, 777
    A = inputs.uniform_s8(M * K, inputs.seed_for(2, 0) + 1)
    B = inputs.uniform_s8(N * K, inputs.seed_for(2, 0) + 2)
    C0 = inputs.uniform_s32(M * N, inputs.seed_for(2, 0) + 3)
    p = _gemm_problem(torch, mg, "ragged_1000x3001x777_acc", M, N, K, A, B, C0=C0, sets=10)
    return Workload("ragged", [p], "TOPS", "int8_gemm_tops",
                    "s8*s8->s32 M,N,K = 1000,3001,777, every pitch misaligned, accumulate=1 onto a seeded int32 C",
                    "hbm", "mip_dense_kernel (+ 1 re-pitch launch for both operands)",
                    "10 copies of the 27 MB problem used in turn (270 MB > L2)")


def build_layouts(torch, mg, n=8192):
    """The same square product under every storage-order combination of A, B and C."""
    A = inputs.uniform_s8(n * n, inputs.seed_for(8, n) + 1)
    B = inputs.uniform_s8(n * n, inputs.seed_for(8, n) + 2)
    dA, dB = _dev_bytes(torch, A), _dev_bytes(torch, B)
    dC = torch.empty(n * n, dtype=torch.int32, device="cuda")
    probs = []
    for ao in (0, 1):
        for bo in (0, 1):
            for cc in (0, 1):
                p = Problem("A%s_B%s_C%s_%d" % ("km"[ao], "kn"[bo], "rc"[cc], n), "layout", 2.0 * n ** 3, 6.0 * n * n)
                p.dims, p.bufs, p.out_bytes = (n, n, n), (dA, dB, dC), 4.0 * n * n
                p.calls = [lambda ao=ao, bo=bo, cc=cc: mg.mipgemm_gemm_ex(0, 0, ao, bo, cc, n, n, n, dA, n, dB, n,
                                                                          dC, n, 0)]
                probs.append(p)
    return Workload("layouts", probs, "TOPS", "int8_gemm_tops",
                    "8192^3 s8*s8->s32 under the eight storage-order combinations (A K-/M-contiguous, "
                    "B K-/N-contiguous, C row-/column-major)", "tensor", "mip_dense_kernel", "operands exceed the L2")


def build_bert(torch, mg, tokens, dequant=False, requant=False):
    probs = []
    t_max = max(tokens)
    for (name, N, K) in inputs.BERT_GEMMS:
        # (the generator is counter based: the activations of fewer tokens are a prefix of those of more)
        A_all = inputs.normal_s8(t_max * K, inputs.seed_for(4, N + K) + 1, 40.0)
        B = inputs.normal_s8(N * K, inputs.seed_for(4, N + K) + 2, 20.0)
        dB = _dev_bytes(torch, B)
        for T in tokens:
            A = A_all[:T * K]
            dA = _dev_bytes(torch, A)
            dC = torch.empty(T * N, dtype=torch.int32, device="cuda")
            p = Problem("%s_T%d" % (name, T), "gemm", 2.0 * T * N * K,
                        T * K + N * K + (1.0 if requant else 4.0) * T * N)
            p.dims, p.ld, p.bufs, p.host = (T, N, K), (K, K, N), (dA, dB, dC), (A, B, None)
            p.out_bytes = (1.0 if requant else 4.0) * T * N
            if requant:     # int8 codes written into the front of the same buffer
                p.kind = "other"
                p.calls = [lambda T=T, N=N, K=K, dA=dA, dB=dB, dC=dC:
                           mg.mipgemm_s8s8s8_requant(T, N, K, dA, K, dB, K, dC, N, 1.25e-3)]
            elif dequant:
                p.kind = "other"
                p.calls = [lambda T=T, N=N, K=K, dA=dA, dB=dB, dC=dC:
                           mg.mipgemm_s8s8f32_dequant(T, N, K, dA, K, dB, K, dC, N, 1.25e-3)]
            else:
                p.calls = [lambda T=T, N=N, K=K, dA=dA, dB=dB, dC=dC:
                           mg.mipgemm_s8s8s32(T, N, K, dA, K, dB, K, dC, N, 0)]
            probs.append(p)
    probs.sort(key=lambda q: q.dims[0])
    return Workload("bert", probs, "TOPS", "int8_gemm_tops",
                    "BERT base/large encoder GEMMs s8*s8->s32 (fused QKV, attention-out, FFN1, FFN2), tokens %s"
                    % list(tokens), "tensor", "mip_dense_kernel", "operands + outputs of one step: 1.6 GB")


def build_resnet(torch, mg, batch, dequant=False, requant=False, x_cache=None):
    """All 53 convolutions (23 distinct shapes x multiplicity).  ``x_cache`` keeps the generated batch-128
    activations of a layer so that a smaller batch (a prefix: the generator is counter based) re-uses them."""
    probs = []
    for li, (cnt, H, W, Cin, Cout, R, S, st, pd) in enumerate(inputs.RESNET50_CONVS):
        Ho = (H + 2 * pd - (R - 1) - 1) // st + 1
        Wo = (W + 2 * pd - (S - 1) - 1) // st + 1
        per_image = H * W * Cin
        if x_cache is not None and li in x_cache and x_cache[li].size >= batch * per_image:
            X = x_cache[li][:batch * per_image]
        else:
            X = inputs.uniform_u8(batch * per_image, inputs.seed_for(3, li) + 1)
            if x_cache is not None:
                x_cache[li] = X
        Wt = inputs.normal_s8(Cout * R * S * Cin, inputs.seed_for(3, li) + 2, 32.0, -127, 127)
        dX, dW = _dev_bytes(torch, X), _dev_bytes(torch, Wt)
        dY = torch.empty(batch * Ho * Wo * Cout, dtype=torch.int32, device="cuda")
        M, K = batch * Ho * Wo, R * S * Cin
        p = Problem("conv%02d_%dx%dx%d_%d_%dx%d_s%d" % (li + 1, H, W, Cin, Cout, R, S, st), "conv",
                    2.0 * M * Cout * K, batch * H * W * Cin + Cout * K + (1.0 if requant else 4.0) * M * Cout)
        p.dims, p.count, p.bufs = (M, Cout, K), cnt, (dX, dW, dY)
        p.geom = (batch, H, W, Cin, Cout, R, S, st, pd, Ho, Wo)
        p.host = (X, Wt, None)
        p.out_bytes = (1.0 if requant else 4.0) * M * Cout
        a = (batch, H, W, Cin, Cout, R, S, st, st, pd, pd, 1, 1)
        if requant:         # uint8 codes (ReLU included) written into the front of the same buffer
            p.kind = "other"
            p.calls = [lambda a=a, dX=dX, dW=dW, dY=dY: mg.mipgemm_conv_u8s8u8_requant(*a, dX, dW, dY, 7.5e-4)]
        elif dequant:
            p.kind = "other"
            p.calls = [lambda a=a, dX=dX, dW=dW, dY=dY: mg.mipgemm_conv_u8s8f32_dequant(*a, dX, dW, dY, 7.5e-4)]
        else:
            p.calls = [lambda a=a, dX=dX, dW=dW, dY=dY: mg.mipgemm_conv_u8s8s32(*a, dX, dW, dY, 0)]
        probs.append(p)
    return Workload("resnet50_b%d" % batch, probs, "TOPS", "int8_conv_tops",
                    "ResNet-50 v1.5 convolutions u8*s8->s32 NHWC, batch %d, 53 layers, lowering included" % batch,
                    "hbm", "mip_dense_kernel (TMA im2col / gathered stem)",
                    "activations + outputs of one step: %.1f GB" % (sum(q.bytes * q.count for q in probs) / 1e9))


def build_paper_b1(torch, mg):
    """The paper's own evaluation setting (Section 7.2): batch 1 -- all 53 ResNet-50 v1.5 convolutions
    plus the final fully connected layer as a matrix-vector product (2048 -> 1000), and the six
    weight GEMMs of one BERT-Large encoder block (Table 5) for one sentence of l = 512 tokens."""
    probs = build_resnet(torch, mg, 1).probs
    K, N = 2048, 1000
    A = inputs.uniform_u8(K, inputs.seed_for(3, 99) + 1)
    B = inputs.normal_s8(N * K, inputs.seed_for(3, 99) + 2, 32.0, -127, 127)
    probs.append(_gemm_problem(torch, mg, "fc_gemv_2048_1000", 1, N, K, A, B, mode="u8"))
    T, d, f = 512, 1024, 4096
    for (name, n, k, cnt) in [("M1-M3_qkv", d, d, 3), ("M9_attn_out", d, d, 1), ("F11_ffn1", f, d, 1), ("F13_ffn2", d, f, 1)]:
        A = inputs.normal_s8(T * k, inputs.seed_for(4, n + k) + 1, 40.0)
        B = inputs.normal_s8(n * k, inputs.seed_for(4, n + k) + 2, 20.0)
        p = _gemm_problem(torch, mg, "bert_large_l512_%s" % name, T, n, k, A, B)
        p.count = cnt
        probs.append(p)
    return Workload("paper_b1", probs, "TOPS", "int8_b1_tops",
                    "the paper's batch-1 setting: ResNet-50 v1.5 (53 convs + FC matrix-vector product) and one "
                    "BERT-Large encoder block, l = 512", "tensor", "mip_dense_kernel",
                    "operands stay L2-resident (batch-1 problems are a few MB): a latency measurement, as in the "
                    "paper's setting")


def build_attention(torch, mg, sentences=8, heads=16, l=512, dh=64):
    """The activation-by-activation products of BERT-Large's attention (paper Table 5): M5, l x l x d/h,
    and M7, d/h x l x l, one per head and sentence, as strided int8 batches."""
    batch = sentences * heads
    probs = []
    for (name, M, N, K) in [("M5_scores", l, l, dh), ("M7_context", l, dh, l)]:
        A = inputs.normal_s8(batch * M * K, inputs.seed_for(4, 900 + K) + 1, 40.0)
        B = inputs.normal_s8(batch * N * K, inputs.seed_for(4, 900 + K) + 2, 40.0)
        dA, dB = _dev_bytes(torch, A), _dev_bytes(torch, B)
        dC = torch.empty(batch * M * N, dtype=torch.int32, device="cuda")
        p = Problem("attention_%s_x%d" % (name, batch), "other", 2.0 * batch * M * N * K,
                    batch * (M * K + N * K + 4.0 * M * N))
        p.dims, p.bufs, p.out_bytes = (M, N, K), (dA, dB, dC), 4.0 * batch * M * N
        p.calls = [lambda M=M, N=N, K=K, dA=dA, dB=dB, dC=dC:
                   mg.mipgemm_batched_s8s8s32(batch, M, N, K, dA, K, M * K, dB, K, N * K, dC, N, M * N, 0)]
        probs.append(p)
    return Workload("attention", probs, "TOPS", "int8_batched_tops",
                    "BERT-Large attention products M5 (512x512x64) and M7 (512x64x512) as strided int8 batches of 128",
                    "hbm", "mip_dense_kernel", "operands exceed the L2")


def build_skinny(torch, mg, rotate_bytes=512 << 20):
    """Decode GEMMs.  Every weight matrix exists in several rotation slots so that a step never finds its
    weights in the L2: slot r holds the seeded matrix with its rows rotated by r (a device-side copy; the
    oracle comparison rotates the host copy the same way)."""
    probs = []
    for (N, K) in inputs.SKINNY_WEIGHTS:
        slots = max(2, -(-rotate_bytes // (N * K)))
        B = inputs.uniform_s8(N * K, inputs.seed_for(5, N + K) + 2)
        d0 = _dev_bytes(torch, B).view(N, K)
        Bs = [d0.reshape(-1)] + [torch.roll(d0, r, 0).reshape(-1).contiguous() for r in range(1, slots)]
        for M in inputs.SKINNY_M:
            A = inputs.uniform_s8(M * K, inputs.seed_for(5, M) + 1)
            dA = _dev_bytes(torch, A)
            dC = torch.empty(M * N, dtype=torch.int32, device="cuda")
            p = Problem("skinny_M%d_%dx%d" % (M, N, K), "skinny", 2.0 * M * N * K, N * K + M * K + 4.0 * M * N)
            p.dims, p.ld, p.bufs, p.host = (M, N, K), (K, K, N), (dA, Bs, dC), (A, B, None)
            p.out_bytes = 4.0 * M * N
            p.calls = [lambda M=M, N=N, K=K, dA=dA, dB=dB, dC=dC:
                       mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 0) for dB in Bs]
            probs.append(p)
    return Workload("skinny", probs, "GB/s", "skinny_gemm_gbs",
                    "decode GEMMs s8*s8->s32, M in %s, weights %s, every weight matrix rotated over >= 512 MB of "
                    "copies" % (inputs.SKINNY_M, inputs.SKINNY_WEIGHTS), "hbm", "mip_skinny_ring_kernel",
                    "weights rotate over >= 512 MB per matrix: never L2-resident")


# --------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Samples SM clock and clock-event reasons through NVML while a timed region runs
    (read-only queries)."""

    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}
    _nv = None
    _handle = None
    _max_sm = None
    _err = None

    @classmethod
    def _open(cls, torch, device_index):
        if cls._handle is not None or cls._err is not None:
            return
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                handle = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            cls._max_sm = int(pynvml.nvmlDeviceGetMaxClockInfo(handle, pynvml.NVML_CLOCK_SM))
            cls._nv, cls._handle = pynvml, handle
        except Exception as exc:  # NVML missing: report that instead of inventing numbers
            cls._err = repr(exc)

    def __init__(self, torch, device_index, period_s=0.003):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.power = [], set(), []
        self.stop_flag = threading.Event()
        self.period_s = period_s
        self._open(torch, device_index)
        self.ok = self._handle is not None

    def _once(self):
        nv, h = self._nv, self._handle
        self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
        try:
            getter = getattr(nv, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                nv.nvmlDeviceGetCurrentClocksThrottleReasons
            mask = int(getter(h))
            for bit, name in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
        except Exception:
            pass
        try:
            self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
        except Exception:
            pass

    def run(self):
        if not self.ok:
            return
        while not self.stop_flag.is_set():
            try:
                self._once()
            except Exception:
                break
            time.sleep(self.period_s)

    def finish(self):
        self.stop_flag.set()
        self.join(timeout=2.0)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "note": "NVML unavailable"}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self._max_sm,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": rnd(max(self.power)) if self.power else None}


# --------------------------------------------------------------------------- timing
def run_step(wl, events=None):
    for j, (p, reps) in enumerate(wl.groups):
        if events is not None:
            events[j][0].record()
        for i in range(reps):
            p.calls[i % len(p.calls)]()
        if events is not None:
            events[j][1].record()
    wl.steps_run += 1


def host_call_cost(torch, mg, wl, passes):
    """Wall-clock microseconds the C-ABI call itself takes on the host (argument checks, planning,
    tensor-map encoding, launch; no synchronisation inside the timed calls), averaged over the launches of
    a step.  The first pass is the cold figure (every shape and pointer seen for the first time)."""
    out = []
    for _ in range(passes):
        torch.cuda.synchronize()
        t = 0.0
        for (p, reps) in wl.groups:
            for i in range(reps):
                fn = p.calls[i % len(p.calls)]
                t0 = time.perf_counter()
                fn()
                t += time.perf_counter() - t0
            if reps * p.ops > 5e11:          # keep the launch queue short behind long kernels
                torch.cuda.synchronize()
        wl.steps_run += 1
        out.append(t / wl.launches_per_step * 1e6)
    torch.cuda.synchronize()
    return out


def time_workload(torch, mg, wl, steps, warmup, eager, world, dist, local_rank, min_region_ms=0.0, detail=True):
    """Warm-up, one CUDA-graph capture of a step, `steps` timed replays bracketed by events and
    synchronisation, clocks sampled during the region; then per-problem times from a second capture that
    carries an event pair per problem (event records between two kernels keep the second from starting its
    prologue under the first one's tail, so they stay out of the timed graph)."""
    res = {}
    host_us = host_call_cost(torch, mg, wl, 1 + max(warmup, 3))
    res["host_us_per_call"] = {"cold": rnd(host_us[0]), "warm": rnd(float(np.median(host_us[1:])))}
    assert mg.mipgemm_device_status() == mg.OK
    graph = None
    count0 = mg.mipgemm_launch_count()
    if not eager:
        graph = torch.cuda.CUDAGraph()
        steps_before = wl.steps_run
        with torch.cuda.graph(graph):
            run_step(wl)
        wl.steps_run = steps_before
        kernels_per_step = mg.mipgemm_launch_count() - count0
        graph.replay()
        wl.steps_run += 1
        torch.cuda.synchronize()
        assert mg.mipgemm_device_status() == mg.OK
        if min_region_ms > 0.0:      # short steps: enough replays for the clock sampler to see the region
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            graph.replay()
            e1.record()
            torch.cuda.synchronize()
            wl.steps_run += 1
            steps = max(steps, int(np.ceil(min_region_ms / max(e0.elapsed_time(e1), 1e-3))))
            steps = min(steps, 4000)
    sampler = ClockSampler(torch, local_rank)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = mg.mipgemm_launch_count()
    sampler.start()
    stream = torch.cuda.current_stream()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    group_ms = [0.0] * len(wl.groups)
    if graph is not None:
        ev0.record(stream)
        for _ in range(steps):
            graph.replay()
        ev1.record(stream)
        torch.cuda.synchronize()
        wl.steps_run += steps
    else:
        eager_events = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                         for _ in wl.groups] for _ in range(steps)]
        ev0.record(stream)
        for s in range(steps):
            run_step(wl, eager_events[s])
        ev1.record(stream)
        torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    res["clocks"] = sampler.finish()
    launches = (kernels_per_step * steps) if graph is not None else (mg.mipgemm_launch_count() - launches0)
    assert mg.mipgemm_device_status() == mg.OK
    elapsed_ms = sharding.max_over_ranks(ev0.elapsed_time(ev1), dist if world > 1 else None,
                                         torch.device("cuda", local_rank))
    detail_reps = 3 if graph is not None else steps
    if graph is not None and detail:
        graph_events = [(torch.cuda.Event(enable_timing=True, external=True),
                         torch.cuda.Event(enable_timing=True, external=True)) for _ in wl.groups]
        graph_detail = torch.cuda.CUDAGraph()
        steps_before = wl.steps_run
        with torch.cuda.graph(graph_detail):
            run_step(wl, graph_events)
        wl.steps_run = steps_before
        for _ in range(detail_reps):
            graph_detail.replay()
            wl.steps_run += 1
            torch.cuda.synchronize()
            for j, (a, b) in enumerate(graph_events):
                group_ms[j] += a.elapsed_time(b)
        del graph_detail
    elif graph is None:
        for s in range(steps):
            for j, (a, b) in enumerate(eager_events[s]):
                group_ms[j] += a.elapsed_time(b)
    per_problem = []
    if detail:
        for j, (p, reps) in enumerate(wl.groups):
            avg = group_ms[j] / (detail_reps * reps)          # ms per launch of this problem
            per_problem.append({"name": p.name, "launches": reps, "us": rnd(avg * 1e3),
                                "tops": rnd(p.ops / (avg * 1e-3) / 1e12), "gbs": rnd(p.bytes / (avg * 1e-3) / 1e9)})
    res.update(steps=steps, elapsed_ms=elapsed_ms, ms_per_step=elapsed_ms / steps, launches=int(launches),
               per_problem=per_problem, launch="eager" if graph is None else "one CUDA graph replay per step")
    del graph
    return res


def roofline_of(wl, res, peaks, probe, write_gbs, world=1):
    """Roofline record of one workload's timed region.  The region holds nothing but the workload's kernels,
    so the dominant kernel's average launch duration is the elapsed time over the launches."""
    sec = res["ms_per_step"] * 1e-3
    tops = wl.step_ops / sec / 1e12
    gbs = wl.step_bytes / sec / 1e9
    int8_burst = peaks["bf16_tflops"] * (NOMINAL_INT8_TOPS / NOMINAL_BF16_TFLOPS)
    int8_sust = peaks["bf16_tflops_sustained"] * (NOMINAL_INT8_TOPS / NOMINAL_BF16_TFLOPS)
    src = peaks["_source"]
    # what a perfect implementation would need: every problem at the slower of its two roofs
    ideal_s = sum(r * max(p.ops / (int8_burst * 1e12), p.bytes / (peaks["hbm_gbs"] * 1e9)) for (p, r) in wl.groups)
    if wl.bound == "tensor":
        roof = {"bound": "tensor", "kernel": wl.kernel, "achieved": rnd(tops, 6), "peak": rnd(int8_burst, 6),
                "unit": "TFLOP/s", "frac": rnd(tops / int8_burst),
                "peak_source": "%s bf16 cuBLAS burst x2 (nominal int8:bf16 ratio)" % src,
                "frac_of_sustained": rnd(tops / int8_sust), "frac_of_nominal_4500": rnd(tops / NOMINAL_INT8_TOPS)}
    else:
        roof = {"bound": "hbm", "kernel": wl.kernel, "achieved": rnd(gbs, 6), "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": rnd(gbs / peaks["hbm_gbs"]),
                "peak_source": "%s copy bandwidth" % src, "frac_of_nominal_8000": rnd(gbs / NOMINAL_HBM_GBS)}
        if write_gbs:
            roof["write_gbs"] = rnd(wl.step_out_bytes / sec / 1e9)
            roof["frac_of_write_rate"] = rnd(wl.step_out_bytes / sec / 1e9 / write_gbs)
    if probe and probe.get("burst_tops"):
        roof["frac_of_i8_probe"] = rnd(tops / probe["burst_tops"])
    roof["tops"], roof["gbs"] = rnd(tops), rnd(gbs)
    roof["frac_of_per_problem_roofs"] = rnd(ideal_s / sec)
    roof["traffic"] = load_traffic(wl.name)
    roof["launches_timed"] = wl.launches_per_step * res["steps"]
    return roof


# --------------------------------------------------------------------------- device-side reference rates
def measure_probe(torch, mg, sustained_s=0.0):
    """The tensor pipe's own int8 rate (tcgen05.mma.kind::i8 on operands resident in shared memory)."""
    import ctypes
    sink = torch.empty(4096, dtype=torch.int32, device="cuda")
    grid, ops = ctypes.c_int(0), ctypes.c_double(0.0)

    def launch(iters):
        st = mg._lib.mipgemm_probe_i8_peak(iters, ctypes.byref(grid), ctypes.byref(ops), sink.data_ptr(),
                                           torch.cuda.current_stream().cuda_stream)
        assert st == mg.OK
    out = {}
    launch(2000)
    torch.cuda.synchronize()
    best = 0.0
    for _ in range(3):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        launch(20000)       # ~ 6 ms
        e1.record()
        torch.cuda.synchronize()
        best = max(best, ops.value / (e0.elapsed_time(e1) * 1e-3) / 1e12)
    out["burst_tops"] = rnd(best, 5)
    if sustained_s > 0:
        n = int(sustained_s / 0.03) + 1
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for _ in range(n // 2):
            launch(100000)
        e0.record()
        for _ in range(n):
            launch(100000)
        e1.record()
        torch.cuda.synchronize()
        out["sustained_tops"] = rnd(n * ops.value / (e0.elapsed_time(e1) * 1e-3) / 1e12, 5)
    assert mg.mipgemm_device_status() == mg.OK
    return out


def measure_write_rate(torch, mg, n=16384):
    """What a kernel can write to HBM per second, over 1 GiB of int32, best of three each: a plain fill
    kernel (torch), the library's zero fill (a K = 0 product) and the library's own output path with next to
    nothing to read (K = 64, N = 2048: the epilogue's TMA tile stores).  The fastest of these is the write
    roof quoted beside the output-bound workloads.  A device memset is listed for context only: it clears
    faster than the copy rate (it does not stream the bytes through the SMs) and is no roof for a kernel."""
    dC = torch.empty(n * n, dtype=torch.int32, device="cuda")
    M, N, K = n * n // 2048, 2048, 64
    dA = torch.zeros(M * K, dtype=torch.int8, device="cuda")
    dB = torch.zeros(N * K, dtype=torch.int8, device="cuda")
    best = {}
    for name, fn in (("fill_kernel", lambda: dC.fill_(0x01020304)),
                     ("k0_zero_fill", lambda: mg.mipgemm_s8s8s32(n, n, 0, 0, 1, 0, 1, dC, n, 0)),
                     ("k64_gemm_store", lambda: mg.mipgemm_s8s8s32(M, N, K, dA, K, dB, K, dC, N, 0)),
                     ("memset", dC.zero_)):
        fn()
        torch.cuda.synchronize()
        t = 1e9
        for _ in range(3):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            t = min(t, e0.elapsed_time(e1))
        best[name] = 4.0 * n * n / (t * 1e-3) / 1e9
    del dC, dA, dB
    return best


# --------------------------------------------------------------------------- oracle comparisons
def sample_rows(M, count, seed):
    """First and last rows plus seeded random ones (sorted, distinct)."""
    if M <= count:
        return np.arange(M)
    rng = np.random.default_rng(seed)
    rows = set([0, M - 1]) | set(int(v) for v in rng.integers(0, M, size=count))
    return np.array(sorted(rows))[:max(count, 2)]


def parity_workload(torch, wl, rows_per_problem=48):
    """Compares what the timed launches left in their output buffers with the CPU oracle: sampled rows
    of every GEMM, one whole image of every convolution layer, every cell of the decode GEMMs.
    Returns {"ok": bool, "checked": text, "oracle_s": seconds}."""
    from oracle import mip_oracle as orc
    ok, cells, t_or = True, 0, 0.0
    bad = []
    for li, p in enumerate(wl.probs):
        if p.kind == "gemm":
            M, N, K = p.dims
            lda, ldb, ldc = p.ld
            A, B, C0 = p.host
            rot = getattr(p, "sets", 1) - 1     # the compared copy holds A and B rotated by this many rows
            if rot:
                A = np.ascontiguousarray(np.roll(A.reshape(M, lda), rot, 0)).reshape(-1)
                B = np.ascontiguousarray(np.roll(B.reshape(N, ldb), rot, 0)).reshape(-1)
            rows = sample_rows(M, rows_per_problem, 17 + M + N)
            got = p.bufs[2].view(-1, ldc)[torch.from_numpy(rows).cuda()][:, :N].cpu().numpy()
            A_rows = np.ascontiguousarray(A.reshape(-1)[:M * lda].reshape(M, lda)[rows, :K])
            t0 = time.perf_counter()
            want = orc.gemm(A_rows, B, len(rows), N, K, ldb=ldb).reshape(len(rows), N)
            t_or += time.perf_counter() - t0
            if p.accumulate:   # the buffer has received the product once per launch since it held C0
                total = C0.reshape(M, ldc)[rows, :N].astype(np.int64) + wl.steps_run * want.astype(np.int64)
                want = (total & 0xFFFFFFFF).astype(np.uint32).view(np.int32)     # (C += wraps modulo 2^32, as documented)
        elif p.kind == "conv":
            batch, H, W, Cin, Cout, R, S, st, pd, Ho, Wo = p.geom
            X, Wt, _ = p.host
            img = (3 * li + 1) % batch
            got = p.bufs[2].view(batch, Ho * Wo * Cout)[img].cpu().numpy().reshape(1, Ho, Wo, Cout)
            Xi = X.reshape(batch, H, W, Cin)[img:img + 1]
            t0 = time.perf_counter()
            want = orc.conv(Xi, Wt.reshape(Cout, R, S, Cin), stride=(st, st), pad=(pd, pd))
            t_or += time.perf_counter() - t0
        elif p.kind == "skinny":
            M, N, K = p.dims
            A, B, _ = p.host
            last = (len(p.calls) - 1)          # the slot the step's last launch of this problem used
            got = p.bufs[2].cpu().numpy().reshape(M, N)
            Bh = np.ascontiguousarray(np.roll(B.reshape(N, K), last, 0))
            t0 = time.perf_counter()
            want = orc.gemm(A, Bh, M, N, K).reshape(M, N)
            t_or += time.perf_counter() - t0
        else:
            continue
        cells += want.size
        if not np.array_equal(got, want):
            ok = False
            bad.append(p.name)
    what = {"gemm": "%d sampled rows of every GEMM" % rows_per_problem, "conv": "one whole image of every layer",
            "skinny": "every cell"}
    kinds = sorted(set(p.kind for p in wl.probs if p.kind in what))
    return {"ok": ok, "checked": "; ".join(what[k] for k in kinds) + " (%d cells)" % cells,
            "oracle_s": rnd(t_or, 3), **({"mismatch": bad[:4]} if bad else {})}


def oracle_sample_rows(problems, frac):
    return [max(1, min(p.dims[0], int(round(p.dims[0] * frac)))) for p in problems]


def time_oracle_sample(problems, frac, compare_with=None):
    """Runs the oracle on the first rows of every GEMM of the workload; returns (seconds, ops, parity).
    If ``compare_with`` maps a problem name to the GPU result, the sampled rows are also
    compared bit for bit."""
    from oracle import mip_oracle as orc
    total_s, total_ops, parity = 0.0, 0.0, None
    for p, r in zip(problems, oracle_sample_rows(problems, frac)):
        M, N, K = p.dims
        A, B = p.host[0], p.host[1]
        t0 = time.perf_counter()
        want = orc.gemm(A[:r * K], B, r, N, K)
        total_s += time.perf_counter() - t0
        total_ops += 2.0 * r * N * K
        if compare_with is not None and p.name in compare_with:
            same = bool(np.array_equal(compare_with[p.name][:r * N], want))
            parity = same if parity is None else (parity and same)
    return total_s, total_ops, parity


def calibrate_fraction(problems, target_s):
    """Sample fraction (of every problem's rows) so the oracle runs for about target_s."""
    from oracle import mip_oracle as orc
    p = problems[min(2, len(problems) - 1)]
    M, N, K = p.dims
    A, B = p.host[0], p.host[1]
    r = min(M, 128)                                    # (enough rows for every oracle thread to get some)
    orc.gemm(A[:r * K], B, r, N, K)                    # builds / warms the oracle
    t0 = time.perf_counter()
    orc.gemm(A[:r * K], B, r, N, K)
    rate = 2.0 * r * N * K / max(time.perf_counter() - t0, 1e-6)
    total = sum(q.ops for q in problems)
    return max(1e-6, min(1.0, target_s * rate / total))


def host_only_square(sizes):
    probs = []
    for n in sizes:
        p = Problem("square_%d" % n, "gemm", 2.0 * n * n * n, 6.0 * n * n)
        p.dims = (n, n, n)
        p.host = (inputs.uniform_s8(n * n, inputs.seed_for(2, n) + 1),
                  inputs.uniform_s8(n * n, inputs.seed_for(2, n) + 2))
        probs.append(p)
    return probs


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores: each step a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import mip_oracle as orc
    sizes = [s for s in inputs.SQUARE_SIZES if s <= args.max_size]
    probs = host_only_square(sizes)
    frac = calibrate_fraction(probs, 60.0 / max(1, args.steps + args.warmup))
    for _ in range(args.warmup):
        time_oracle_sample(probs, frac)
    secs, ops = 0.0, 0.0
    for _ in range(args.steps):
        s, o, _p = time_oracle_sample(probs, frac)
        secs += s
        ops += o
    value = ops / secs / 1e12
    rows = oracle_sample_rows(probs, frac)
    sample = "first rows of every sweep member: " + ", ".join(
        "%d of %d" % (r, p.dims[0]) for r, p in zip(rows, probs))
    line = {
        "impl": "reference", "metric": "int8_gemm_tops", "value": value, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": secs / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": "square s8*s8->s32 sweep M=N=K in %s (sampled rows per step)" % sizes},
        "cpu_baseline": {"value": value, "unit": "TOPS", "cores": orc.threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- end to end
def measure_e2e(torch, mg, wl, steps, world, dist, local_rank):
    """The square sweep through the host-buffer entry point (pinned host memory, copies inside the timed
    region), and beside it what the host link alone does with the same bytes: plain pinned copies of the
    step's operands (host to device) and results (device to host), each direction alone and both at once."""
    pinned = []
    for p in wl.probs:
        n = p.dims[0]
        hA = torch.from_numpy(p.host[0].view(np.uint8)).pin_memory()
        hB = torch.from_numpy(p.host[1].view(np.uint8)).pin_memory()
        hC = torch.empty(n * n, dtype=torch.int32).pin_memory()
        pinned.append((n, hA, hB, hC, p))
    h2d = sum(2 * n * n for (n, *_r) in pinned)
    d2h = sum(4 * n * n for (n, *_r) in pinned)

    def e2e_step():
        for (n, hA, hB, hC, _p) in pinned:
            mg.mipgemm_host_s8s8s32(n, n, n, hA, n, hB, n, hC, n, 0)

    e2e_step()
    e2e_steps = max(3, min(steps, 7))
    per_step = []
    for _ in range(e2e_steps):      # (every host call synchronises its stream before it returns)
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        t0 = time.perf_counter()
        e2e_step()
        torch.cuda.synchronize()
        per_step.append(sharding.max_over_ranks(time.perf_counter() - t0, dist if world > 1 else None,
                                                torch.device("cuda", local_rank)))
    # the host path's results against the device path's (already compared with the oracle)
    same = all(bool(torch.equal(hC, p.bufs[2].cpu())) for (_n, _a, _b, hC, p) in pinned)

    # plain copies of the same bytes
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

    def copies(do_in, do_out):
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for (n, hA, hB, hC, p) in pinned:
            if do_in:
                with torch.cuda.stream(s_in):
                    p.bufs[0].copy_(hA, non_blocking=True)
                    p.bufs[1].copy_(hB, non_blocking=True)
            if do_out:
                with torch.cuda.stream(s_out):
                    hC.copy_(p.bufs[2], non_blocking=True)
        torch.cuda.synchronize()
        return time.perf_counter() - t0
    copies(True, True)
    t_in = min(copies(True, False) for _ in range(3))
    t_out = min(copies(False, True) for _ in range(3))
    t_both = min(copies(True, True) for _ in range(3))
    # The host link of these boxes is shared with other tenants: single steps stall by 0.2-2 s now and
    # then (with every build).  The median step is reported; the mean is kept beside it.
    e2e_s = sorted(per_step)[len(per_step) // 2]
    return {"value": rnd(world * wl.step_ops / e2e_s / 1e12, 6), "unit": "TOPS", "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": rnd(e2e_s * 1e3, 5), "steps": e2e_steps,
            "stat": "median step", "ms_per_step_mean": rnd(sum(per_step) / len(per_step) * 1e3, 5),
            "ms_per_step_best": rnd(min(per_step) * 1e3, 5),
            "link": {"h2d_gbs": rnd(h2d / t_in / 1e9), "d2h_gbs": rnd(d2h / t_out / 1e9),
                     "both_directions_ms": rnd(t_both * 1e3, 5),
                     "what": "pinned cudaMemcpyAsync of the same operands / results, best of 3"},
            "e2e_frac_of_link": rnd(t_both / e2e_s),
            "matches_device_path": same,
            "api": "mipgemm_host_s8s8s32 (pinned host buffers; blocks of C pipelined over three streams)"}


# --------------------------------------------------------------------------- main arm
SECONDARY = ["gemm512", "ragged", "bert", "resnet50_b32", "resnet50_b128", "skinny_const_weights", "skinny"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all",
                    choices=["all", "square", "gemm512", "ragged", "bert", "resnet", "skinny", "paper_b1",
                             "attention", "layouts"],
                    help="all: the square sweep as the headline plus every other configuration under 'workloads'")
    ap.add_argument("--max-size", type=int, default=16384, help="largest member of the square sweep")
    ap.add_argument("--batch", type=int, default=32, help="resnet batch")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--detail", action="store_true", help="per-problem timings in the JSON line and on stderr")
    ap.add_argument("--eager", action="store_true", help="plain launches instead of CUDA-graph replay")
    ap.add_argument("--dequant", action="store_true",
                    help="bert/resnet: call the fused-dequantisation entry points (float32 = scale * sum)")
    ap.add_argument("--no-weights-hint", action="store_true",
                    help="skinny: do not declare the weights constant (no early weight fetch across launches)")
    ap.add_argument("--requant", action="store_true",
                    help="bert/resnet: call the requantising entry points (8-bit codes = sat(rne(scale * sum)))")
    ap.add_argument("--only", default="", help="keep only problems whose name contains this text (for profiling)")
    ap.add_argument("--sustained-s", type=float, default=1.5,
                    help="all: seconds of back-to-back replays of the headline step for the power-capped figure")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    from paper_2506_11728_b200 import build as _build
    _build.build_library()
    from paper_2506_11728_b200 import binding as mg

    peaks = load_peaks()
    headline_name = "square" if args.workload == "all" else args.workload
    everything = args.workload == "all"
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline and headline_name == "square"
    common = dict(eager=args.eager, world=world, dist=dist, local_rank=local_rank)

    # one small call absorbs the library's per-device set-up, so that "cold" host times below mean
    # "first call with these shapes and pointers", not "first call of the process"
    tiny = torch.zeros(256 * 256, dtype=torch.int8, device="cuda")
    tiny_c = torch.empty(256 * 256, dtype=torch.int32, device="cuda")
    mg.mipgemm_s8s8s32(256, 256, 256, tiny, 256, tiny, 256, tiny_c, 256, 0)
    torch.cuda.synchronize()

    # what the Python binding alone costs per call (an empty problem returns before any CUDA call): the
    # host_us_per_call figures below include it
    t0 = time.perf_counter()
    for _ in range(2000):
        mg.mipgemm_s8s8s32(0, 256, 256, tiny, 256, tiny, 256, tiny_c, 256, 0)
    binding_us = (time.perf_counter() - t0) / 2000 * 1e6

    probe = measure_probe(torch, mg) if everything else None
    write = measure_write_rate(torch, mg) if everything else None
    write_gbs = max(v for k, v in write.items() if k != "memset") if write else None

    def build(name):
        if name == "square":
            return build_square(torch, mg, [s for s in inputs.SQUARE_SIZES if s <= args.max_size])
        if name == "gemm512":
            return build_gemm512(torch, mg)
        if name == "ragged":
            return build_ragged(torch, mg)
        if name == "bert":
            return build_bert(torch, mg, inputs.BERT_TOKENS, args.dequant, args.requant)
        if name == "resnet":
            return build_resnet(torch, mg, args.batch, args.dequant, args.requant)
        if name == "attention":
            return build_attention(torch, mg)
        if name == "layouts":
            return build_layouts(torch, mg)
        if name == "paper_b1":
            return build_paper_b1(torch, mg)
        return build_skinny(torch, mg)

    # ---- headline workload
    wl = build(headline_name)
    if headline_name == "skinny" and not args.no_weights_hint:
        mg.mipgemm_set_weights_constant(1)      # decode: the weights are never written between calls
        wl.text += ", weights declared constant (mipgemm_set_weights_constant)"
    if args.requant and headline_name in ("bert", "resnet"):
        wl.text += ", fused requantisation to 8-bit codes"
    elif args.dequant and headline_name in ("bert", "resnet"):
        wl.text += ", fused dequantisation to float32"
    if args.only:
        keep = [p for p in wl.probs if args.only in p.name]
        if not keep:
            raise SystemExit("--only matched no problem")
        wl = Workload(wl.name, keep, wl.unit, wl.metric, wl.text + " [only: %s]" % args.only, wl.bound, wl.kernel,
                      wl.l2_note)

    res = time_workload(torch, mg, wl, args.steps, args.warmup, **common)
    ms_per_step = res["ms_per_step"]
    value = world * (wl.step_ops / 1e12 if wl.unit == "TOPS" else wl.step_bytes / 1e9) / (ms_per_step * 1e-3)
    roofline = roofline_of(wl, res, peaks, probe, write_gbs)
    if args.detail and rank == 0:
        for d in res["per_problem"]:
            sys.stderr.write("%-40s %10.1f us %9.1f TOPS %9.1f GB/s\n" % (d["name"], d["us"], d["tops"], d["gbs"]))
    headline_parity = parity_workload(torch, wl) if (rank == 0 and not args.no_cpu_baseline) else None

    # ---- the same step replayed for seconds: the power-capped figure, with time x clock beside it
    sustained = None
    if everything and args.sustained_s > 0:
        n_long = max(args.steps, int(args.sustained_s * 1e3 / ms_per_step))
        r2 = time_workload(torch, mg, wl, n_long, 0, detail=False, **common)
        sustained = {"steps": r2["steps"], "ms_per_step": rnd(r2["ms_per_step"], 5),
                     "value": rnd(world * wl.step_ops / (r2["ms_per_step"] * 1e-3) / 1e12, 6), "unit": "TOPS",
                     "clocks": r2["clocks"],
                     "ms_x_ghz": rnd(r2["ms_per_step"] * (r2["clocks"]["sm_mhz"] or 0) / 1e3, 5),
                     "short_region_ms_x_ghz": rnd(ms_per_step * (res["clocks"]["sm_mhz"] or 0) / 1e3, 5)}

    # ---- end to end through the host-buffer entry point (pinned host memory, copies timed); with several
    # ranks all of them run it at the same time (they share the host's links) and the slowest rank counts
    e2e = None
    if headline_name == "square" and not args.no_e2e:
        e2e = measure_e2e(torch, mg, wl, args.steps, world, dist, local_rank)

    # ---- the CPU oracle on a bounded sample of the same workload, same run
    cpu = None
    if want_cpu:
        from oracle import mip_oracle as orc
        frac = calibrate_fraction(wl.probs, 24.0)
        gpu_rows = {}
        for p, r in zip(wl.probs, oracle_sample_rows(wl.probs, frac)):
            gpu_rows[p.name] = p.bufs[2][:r * p.dims[1]].cpu().numpy()
        secs, ops, parity = time_oracle_sample(wl.probs, frac, compare_with=gpu_rows)
        rows = oracle_sample_rows(wl.probs, frac)
        cpu = {"value": rnd(ops / secs / 1e12), "unit": "TOPS", "cores": orc.threads(), "kind": "oracle",
               "sample": "first rows of every sweep member (%s), %.1f s of CPU time" % (
                   ", ".join("%d/%d" % (r, p.dims[0]) for r, p in zip(rows, wl.probs)), secs),
               "gpu_rows_match_oracle": parity}
    headline_text, headline_l2, headline_lps = wl.text, wl.l2_note, wl.launches_per_step
    headline_metric, headline_unit = wl.metric, wl.unit
    headline_launches = res["launches"]
    total_launches = headline_launches
    del wl
    torch.cuda.empty_cache()

    # ---- every other configuration of the benchmark definition, same protocol
    workloads = {}
    if everything:
        x_cache = {}
        for name in SECONDARY:
            if name == "resnet50_b128":
                w2 = build_resnet(torch, mg, 128, x_cache=x_cache)
            elif name == "resnet50_b32":
                for li, (cnt, H, W, Cin, *_r) in enumerate(inputs.RESNET50_CONVS):   # batch 32 = a prefix of batch 128
                    x_cache[li] = inputs.uniform_u8(128 * H * W * Cin, inputs.seed_for(3, li) + 1)
                w2 = build_resnet(torch, mg, 32, x_cache=x_cache)
            elif name.startswith("skinny"):
                w2 = build_skinny(torch, mg)
                mg.mipgemm_set_weights_constant(1 if name == "skinny_const_weights" else 0)
                if name == "skinny_const_weights":
                    w2.text += ", weights declared constant (mipgemm_set_weights_constant)"
                w2.name = name
            else:
                w2 = build(name)
            r = time_workload(torch, mg, w2, args.steps, args.warmup, min_region_ms=150.0, detail=args.detail,
                              **common)
            mg.mipgemm_set_weights_constant(0)
            v = world * (w2.step_ops / 1e12 if w2.unit == "TOPS" else w2.step_bytes / 1e9) / (r["ms_per_step"] * 1e-3)
            entry = {"value": rnd(v, 6), "unit": w2.unit, "ms_per_step": rnd(r["ms_per_step"], 5),
                     "steps": r["steps"], "launches_per_step": w2.launches_per_step,
                     "roofline": roofline_of(w2, r, peaks, probe, write_gbs), "clocks": r["clocks"],
                     "host_us_per_call": r["host_us_per_call"], "config": w2.text}
            if rank == 0 and not args.no_cpu_baseline:
                entry["parity"] = parity_workload(torch, w2)
            if args.detail:
                entry["per_problem"] = r["per_problem"]
            workloads[name] = entry
            total_launches += r["launches"]
            del w2
            torch.cuda.empty_cache()
        del x_cache
        probe.update(measure_probe(torch, mg, sustained_s=1.0))      # (last: it heats the chip)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": headline_metric, "value": value, "unit": headline_unit, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "config": {"workload": headline_text,
                   "l2": headline_l2 + ("; every buffer is evicted between two uses" if "exceed" in headline_l2 else ""),
                   "launches_per_step": headline_lps, "launch": res["launch"]},
        "clocks": res["clocks"],
        "e2e": e2e,
        "gpu_launches": int(headline_launches),
        "roofline": roofline,
        "cpu_baseline": cpu,
        "host_us_per_call": dict(res["host_us_per_call"], binding_only=rnd(binding_us),
                                 what="wall clock of the C-ABI call through the Python binding, no synchronisation; "
                                      "cold = first call with these arguments, warm = repeated (plan and tensor maps "
                                      "cached); binding_only = the same binding on an empty problem"),
    }
    if headline_parity is not None:
        line["parity"] = headline_parity
    if sustained is not None:
        line["sustained"] = sustained
    if everything:
        line["reference_rates"] = {"i8_probe": probe, "write_gbs": {k: rnd(v) for k, v in write.items()},
                                   "what": "measured in this process: tcgen05.mma.kind::i8 issue probe (TOPS); what a "
                                           "kernel writes to HBM over 1 GiB (GB/s; the fastest but the memset is the "
                                           "write roof of frac_of_write_rate)"}
        line["workloads"] = workloads
        line["gpu_launches_all_workloads"] = int(total_launches)
    if args.detail:
        line["per_problem"] = res["per_problem"]
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
