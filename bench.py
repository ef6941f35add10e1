#!/usr/bin/env python
"""Benchmark of the FB4 online activation quantizer on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one plain FB4 quantization (fb4_quantize) of the 75600 x 12288 bf16 activation tensor
(the largest workload; 1.86 GB in, so every step streams from HBM, far beyond the 126 MB L2).
`value` is algorithmic GB/s (2 B read + 0.5 B codes + 2 B per 32-element block of metadata per
element) over all ranks; with N > 1 every rank quantizes its own tensor of that shape (no
data-path collective; weak scaling).  The other paths of the library (SeDA, decomposition,
decode, the smaller tensor) are timed the same way and reported under "variants".  One JSON
line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "fb4_quantize_throughput"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel on this workload, from the
# ncu capture summarised in profiles/fb4_quantize_flat_c5_plain_dram_bytes.md (1 858 046 464 B read +
# 499 021 056 B written).  The capture's date and the kernel's register count travel with it in the bench line,
# so that a constant that has outlived the kernel shows; set it back to None whenever that kernel changes.
NCU_TRAFFIC_BYTES = 2357105152
NCU_TRAFFIC_SOURCE = {"profile": "profiles/fb4_quantize_flat_c5_plain_dram_bytes.md", "captured": "2026-11-30",
                      "kernel": "fb4_quantize_flat_kernel<0,0,0,0,0,0>", "registers_per_thread": 115}


def algorithmic_bytes(T: int, C: int, B: int = 32, n_res_rows: int = 0, seda: bool = False,
                      decomposed: bool = False) -> float:
    b = T * C * (2 + 0.5) + T * (C // B) * 2
    if seda:
        b += 4 * T
    if decomposed:
        b += n_res_rows * (C * 0.5 + (C // B) * 2) + 4 * T + 4 * n_res_rows
    return float(b)


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
                 "sw_power_cap": 0x4, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.001)   # the timed region can be a few milliseconds long

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def visible_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def time_steps(fn, steps: int, warmup: int, torch, barrier=None):
    """W untimed calls, then K calls timed with CUDA events on the current stream (per-launch
    events too); returns (total ms, list of per-call ms)."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    if barrier:
        barrier()
        torch.cuda.synchronize()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
    ev[0].record()
    for i in range(steps):
        fn()
        ev[i + 1].record()
    torch.cuda.synchronize()
    if barrier:
        barrier()
    per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
    return ev[0].elapsed_time(ev[steps]), per


def run_reference(args):
    """The CPU oracle, as it stands, on the host cores, on the same workload and metric: each step is the whole
    tensor where the run then stays within a few minutes, else a bounded row sample of it."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import fb4_oracle as orc
    from paper_2603_02883_b200 import synth
    w = synth.workloads()["c5_plain"]
    fbk = synth.STANDIN_FORMATBOOK
    # The whole tensor per step when the oracle's speed on this host lets warm-up plus timed steps end within
    # about 200 s; else the first rows of it that do.  The speed is taken from an untimed pass over 4096 rows.
    probe = synth.activation_rows(w, 0, 4096)
    orc.quantize(probe, fbk)
    t0 = time.perf_counter()
    orc.quantize(probe, fbk)
    rows_per_s = 4096 / (time.perf_counter() - t0)
    rows = int(rows_per_s * 200.0 / max(1, args.steps + args.warmup))
    rows = w.T if rows >= w.T else max(4096, rows // 64 * 64)
    bits = synth.activation(w) if rows == w.T else synth.activation_rows(w, 0, rows)
    for _ in range(args.warmup):
        orc.quantize(bits, fbk)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.quantize(bits, fbk)
    dt = (time.perf_counter() - t0) / args.steps
    gbs = algorithmic_bytes(rows, w.C) / dt / 1e9
    cores = os.cpu_count()
    sample = (f"all {w.T} rows of the 75600x12288 tensor per step" if rows == w.T
              else f"first {rows} of {w.T} rows of the 75600x12288 tensor per step")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "gelem_per_s": rows * w.C / dt / 1e9,
        "config": {"workload": f"plain FB4 quantize, {w.T}x{w.C} bf16 (config-5 tensor), block 32, "
                               "full formatbook, two-stage selection",
                   "per_gpu_tokens": w.T, "channels": w.C, "block_size": 32, "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


class Ops:
    """Every library path on one resident tensor: name -> (callable, algorithmic bytes per call).
    Buffers are allocated on first use and kept (the decoded fp32 tensor alone is 3.7 GB)."""

    def __init__(self, q, x, w, torch, fb4, synth):
        self.q, self.x, self.w, self.torch, self.fb4, self.synth = q, x, w, torch, fb4, synth
        self.T, self.C, self.B = w.T, w.C, 32
        self._buf = {}

    def buf(self, name, shape, dtype):
        if name not in self._buf:
            self._buf[name] = self.torch.empty(shape, dtype=dtype, device="cuda")
        return self._buf[name]

    def drop(self, name):
        self._buf.pop(name, None)

    def extras(self):
        if "extras" not in self._buf:
            w, torch, synth = self.w, self.torch, self.synth
            big = synth.Workload(**{**w.__dict__, "decomposed": True, "score_seed": 4, "seda": True,
                                    "n_clusters": 256 if w.T > 40000 else 64, "cluster_seed": 4})
            cid_np, mask_np = synth.clusters(big)
            self._buf["extras"] = dict(
                tile=big.tile, n_sal=-(-w.T // big.tile), score=torch.from_numpy(synth.scores(big)).cuda(),
                cid=torch.from_numpy(cid_np).cuda(), cmask=torch.from_numpy(mask_np.view(np.int32)).cuda())
        return self._buf["extras"]

    def get(self, name):
        q, x, T, C, B, torch, fb4 = self.q, self.x, self.T, self.C, self.B, self.torch, self.fb4
        codes = self.buf("codes", (T, C // 2), torch.uint8)
        meta = self.buf("meta", (T, C // B), torch.int16)
        if name == "plain":
            return (lambda: fb4.fb4_quantize(q.ctx, x, T, C, C, codes, meta)), algorithmic_bytes(T, C)
        if name == "plain_block16":
            if "q16" not in self._buf:
                self._buf["q16"] = fb4.Fb4(device=torch.cuda.current_device(), block_size=16)
            q16 = self._buf["q16"]
            meta16 = self.buf("meta16", (T, C // 16), torch.int16)
            return (lambda: fb4.fb4_quantize(q16.ctx, x, T, C, C, codes, meta16)), T * C * 2.5 + T * (C // 16) * 2
        if name in ("plain_every_element_a_group", "plain_all_dialects_scored"):
            # the two other selection settings of the paper's Table 2 comparison: num_groups = block, select_mode 1
            key = "qg" if name == "plain_every_element_a_group" else "qa"
            if key not in self._buf:
                self._buf[key] = fb4.Fb4(device=torch.cuda.current_device(), num_groups=32) if key == "qg" else \
                    fb4.Fb4(device=torch.cuda.current_device(), select_mode=1)
            qs = self._buf[key]
            return (lambda: fb4.fb4_quantize(qs.ctx, x, T, C, C, codes, meta)), algorithmic_bytes(T, C)
        if name == "quantize_mxfp8_tiled_scales":
            e8 = self.buf("e4m3", (T, C), torch.uint8)
            sc = self.buf("sf", (fb4.fb4_mxfp8_scale_bytes(T, C, 1),), torch.uint8)
            return (lambda: fb4.fb4_quantize_mxfp8(q.ctx, x, T, C, C, None, None, 0, e8, sc, 1)), \
                T * C * 3.0 + T * (C // B)
        if name == "affine_plus_quantize":
            # modulation y = x * (1 + scale_c) + shift_c fused in front of the quantizer
            gen = torch.Generator(device="cuda").manual_seed(7)
            sc = (0.5 * torch.randn(C, device="cuda", generator=gen)).to(torch.bfloat16)
            sh = torch.randn(C, device="cuda", generator=gen).to(torch.bfloat16)
            self._buf["affine"] = (sc, sh)
            return (lambda: fb4.fb4_quantize_affine(q.ctx, x, T, C, C, sc, sh, 1, None, None, 0, codes, meta)), \
                algorithmic_bytes(T, C) + 4 * C
        if name == "layernorm_plus_quantize":
            # LayerNorm statistics + modulation y = n * (1 + scale_c) + shift_c fused in front of the quantizer
            gen = torch.Generator(device="cuda").manual_seed(7)
            sc = (0.5 * torch.randn(C, device="cuda", generator=gen)).to(torch.bfloat16)
            sh = torch.randn(C, device="cuda", generator=gen).to(torch.bfloat16)
            self._buf["layernorm"] = (sc, sh)
            return (lambda: fb4.fb4_quantize_layernorm(q.ctx, x, T, C, C, sc, sh, 1, 1e-6, None, None, 0, codes, meta)), \
                algorithmic_bytes(T, C) + 4 * C
        if name == "affine_plus_quantize_mxfp8":
            gen = torch.Generator(device="cuda").manual_seed(7)
            sc_v = (0.5 * torch.randn(C, device="cuda", generator=gen)).to(torch.bfloat16)
            sh_v = torch.randn(C, device="cuda", generator=gen).to(torch.bfloat16)
            self._buf["affine_mx"] = (sc_v, sh_v)
            e8 = self.buf("e4m3", (T, C), torch.uint8)
            sf = self.buf("sf", (fb4.fb4_mxfp8_scale_bytes(T, C, 1),), torch.uint8)
            return (lambda: fb4.fb4_quantize_affine_mxfp8(q.ctx, x, T, C, C, sc_v, sh_v, 1, None, None, 0, e8, sf, 1)), \
                T * C * 3.0 + T * (C // B) + 4 * C
        if name == "plain_f32":
            xf = self.buf("x32", (T, C), torch.float32)
            xf.copy_(x)
            return (lambda: fb4.fb4_quantize_f32(q.ctx, xf, T, C, C, codes, meta)), T * C * 4.5 + T * (C // B) * 2
        ex = self.extras()
        n_sal, tile, cid, cmask, score = ex["n_sal"], ex["tile"], ex["cid"], ex["cmask"], ex["score"]
        rc = self.buf("rc", (n_sal, C // 2), torch.uint8)
        rm = self.buf("rm", (n_sal, C // B), torch.int16)
        sal = self.buf("sal", (n_sal,), torch.int32)
        if name == "seda":
            return (lambda: fb4.fb4_quantize_seda(q.ctx, x, T, C, C, cid, cmask, cmask.numel(), codes, meta)), \
                algorithmic_bytes(T, C, seda=True)
        if name == "decomposed":
            return (lambda: fb4.fb4_quantize_decomposed(q.ctx, x, T, C, C, score, tile, None, None, 0, codes, meta,
                                                        sal, rc, rm)), \
                algorithmic_bytes(T, C, n_res_rows=n_sal, decomposed=True)
        if name == "decomposed_given_set":
            # salient set given by the caller (reused from an earlier step / global top-k reading)
            fb4.fb4_select_salient_topk(q.ctx, score, T, n_sal, sal)
            return (lambda: fb4.fb4_quantize_decomposed_idx(q.ctx, x, T, C, C, sal, n_sal, None, None, 0, codes, meta,
                                                            rc, rm)), \
                algorithmic_bytes(T, C, n_res_rows=n_sal, decomposed=True) - 4 * T
        if name == "decomposed_seda":
            return (lambda: fb4.fb4_quantize_decomposed(q.ctx, x, T, C, C, score, tile, cid, cmask, cmask.numel(),
                                                        codes, meta, sal, rc, rm)), \
                algorithmic_bytes(T, C, n_res_rows=n_sal, seda=True, decomposed=True)
        if name == "quantize_mxfp8_decomposed_seda":
            # the whole configuration (decomposition + SeDA) straight to two MXFP8 operands
            e8 = self.buf("e4m3", (T, C), torch.uint8)
            sc = self.buf("sf", (fb4.fb4_mxfp8_scale_bytes(T, C, 1),), torch.uint8)
            r8 = self.buf("res_e4m3", (n_sal, C), torch.uint8)
            rs = self.buf("res_sf", (fb4.fb4_mxfp8_scale_bytes(n_sal, C, 1),), torch.uint8)
            return (lambda: fb4.fb4_quantize_mxfp8_decomposed(q.ctx, x, T, C, C, score, tile, sal, 0, cid, cmask,
                                                              cmask.numel(), e8, sc, r8, rs, 1)), \
                T * C * 3.0 + T * (C // B) + n_sal * (C + C // B + 4) + 8 * T
        # the decode ops read what a decomposed quantization left in codes/meta/sal/rc/rm
        fb4.fb4_quantize_decomposed(q.ctx, x, T, C, C, score, tile, None, None, 0, codes, meta, sal, rc, rm)
        plain_bytes = T * C * 0.5 + T * (C // B) * 2
        res_bytes = n_sal * (C * 0.5 + (C // B) * 2) + 4 * n_sal
        if name == "to_mxfp8_tiled_scales":
            e8 = self.buf("e4m3", (T, C), torch.uint8)
            sc = self.buf("sf", (fb4.fb4_mxfp8_scale_bytes(T, C, 1),), torch.uint8)
            return (lambda: fb4.fb4_to_mxfp8(q.ctx, codes, meta, T, C, e8, sc, 1)), \
                plain_bytes + T * C + T * (C // B)
        if name == "dequantize_f32_decomposed":
            out = self.buf("out32", (T, C), torch.float32)
            return (lambda: fb4.fb4_dequantize(q.ctx, codes, meta, T, C, sal, n_sal, rc, rm, out, 0)), \
                plain_bytes + res_bytes + T * C * 4
        if name == "dequantize_f32_plain":
            out = self.buf("out32", (T, C), torch.float32)
            return (lambda: fb4.fb4_dequantize(q.ctx, codes, meta, T, C, None, 0, None, None, out, 0)), \
                plain_bytes + T * C * 4
        if name == "dequantize_bf16_plain":
            out = self.buf("out16", (T, C), torch.bfloat16)
            return (lambda: fb4.fb4_dequantize(q.ctx, codes, meta, T, C, None, 0, None, None, out, 1)), \
                plain_bytes + T * C * 2
        if name == "dequantize_f16_plain":
            out = self.buf("out16", (T, C), torch.bfloat16)
            return (lambda: fb4.fb4_dequantize(q.ctx, codes, meta, T, C, None, 0, None, None, out, 2)), \
                plain_bytes + T * C * 2
        if name == "dequantize_bf16_decomposed":
            out = self.buf("out16", (T, C), torch.bfloat16)
            return (lambda: fb4.fb4_dequantize(q.ctx, codes, meta, T, C, sal, n_sal, rc, rm, out, 1)), \
                plain_bytes + res_bytes + T * C * 2
        raise KeyError(name)


OP_NAMES = ["plain", "plain_block16", "plain_every_element_a_group", "plain_all_dialects_scored", "plain_f32", "affine_plus_quantize", "layernorm_plus_quantize", "seda", "decomposed", "decomposed_given_set", "decomposed_seda", "dequantize_f32_plain", "dequantize_f32_decomposed",
            "dequantize_bf16_plain", "dequantize_bf16_decomposed", "dequantize_f16_plain", "to_mxfp8_tiled_scales",
            "quantize_mxfp8_tiled_scales", "quantize_mxfp8_decomposed_seda", "affine_plus_quantize_mxfp8"]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c5_plain", help="c5_plain (default) or c2 (smaller tensor, for profiling)")
    ap.add_argument("--op", default="plain", choices=OP_NAMES,
                    help="library path timed as the step (default: plain fb4_quantize, the headline metric)")
    ap.add_argument("--generic-kernel", action="store_true",
                    help="force the generic quantize kernel (what the packed, TMA-staged kernel is compared with)")
    ap.add_argument("--no-variants", action="store_true", help="time only the step")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sustained-steps", type=int, default=1500,
                    help="length of the clock-binned run of the step (0 = skip)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":
        return run_reference(args)

    import torch
    from paper_2603_02883_b200 import fb4, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the quantizer has no CPU path")
    torch.cuda.set_device(local_rank)
    barrier = None
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        barrier = dist.barrier

    ws = synth.workloads()
    w = ws[args.workload]
    if world > 1:   # every rank its own tensor of the same shape
        w = synth.Workload(**{**w.__dict__, "seed": w.seed + 1000 * rank})
    bits = synth.activation(w)
    x = torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)
    q = fb4.Fb4(device=local_rank)
    if args.generic_kernel:
        q.set_kernel_variant(1)
    T, C, B = w.T, w.C, 32
    ops = Ops(q, x, w, torch, fb4, synth)
    step, alg = ops.get(args.op)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    l0 = q.launch_count
    with ClockSampler(visible_index(local_rank)) as clk:
        total_ms, per = time_steps(step, args.steps, 0, torch, barrier)
    launches = q.launch_count - l0
    variant = q.last_variant
    t = torch.tensor([total_ms], dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    total_ms = float(t.item())
    ms = total_ms / args.steps
    value = world * alg / (ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    kernel_ms = float(np.mean(per))
    achieved = alg / (kernel_ms * 1e-3) / 1e9
    tensor_name = "config-5" if args.workload == "c5_plain" else args.workload
    op_text = "plain FB4 quantize" if args.op == "plain" else f"FB4 {args.op}"

    out = {
        "metric": METRIC if args.op == "plain" else f"fb4_{args.op}_throughput",
        "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "gelem_per_s": world * T * C / (ms * 1e-3) / 1e9,
        "frac_hbm_measured": value / world / peak, "frac_hbm_nominal_8000": value / world / 8000.0,
        "config": {"workload": f"{op_text}, {T}x{C} bf16 ({tensor_name} tensor), block 32, "
                               "full formatbook, two-stage selection",
                   "per_gpu_tokens": T, "channels": C, "block_size": B, "kernel_variant": variant,
                   "l2": "input 1.86 GB per step, larger than L2; no flush needed" if T * C * 2 > 2.5e8
                         else "input larger than L2 only marginally"},
        "gpu_launches": launches,
        "clocks": clk.summary(),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": NCU_TRAFFIC_BYTES if (args.op == "plain" and args.workload == "c5_plain"
                                                      and not args.generic_kernel) else None,
                     "traffic_source": NCU_TRAFFIC_SOURCE if (args.op == "plain" and args.workload == "c5_plain"
                                                                and not args.generic_kernel) else None,
                     "peak_kind": f"{peak_kind} copy bandwidth",
                     "kernel": f"fb4 {args.op} ({variant})", "algorithmic_bytes_per_launch": alg,
                     "launch_ms_mean": kernel_ms, "launch_ms_min": float(np.min(per))},
    }

    if rank == 0 and args.op == "plain" and not args.no_variants:
        out["quality"] = quality_report(ops, torch, fb4)
    if rank == 0 and not args.no_variants:
        out["variants"] = run_variants(ops, args, torch, fb4, synth, peak)
    if rank == 0 and world == 1 and args.sustained_steps > 0:
        out["sustained"] = run_sustained(step, alg, args.sustained_steps, visible_index(local_rank), torch, peak)
    del ops
    if not args.no_e2e:
        e2e = run_e2e(q, bits, w, args, torch, fb4, barrier)
        if world > 1:
            t = torch.tensor([e2e["seconds_per_step"]], dtype=torch.float64, device="cuda")
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            e2e["seconds_per_step"] = float(t.item())
        e2e["value"] = world * algorithmic_bytes(T, C) / e2e["seconds_per_step"] / 1e9
        out["e2e"] = e2e
    if rank == 0 and not args.no_cpu_baseline:
        out["cpu_baseline"] = run_cpu_baseline(w, synth)
    if rank == 0 and world == 1 and not args.no_variants:
        out["c_abi_host_cost"] = run_host_cost()
    if rank == 0:
        print(json.dumps(out))
    q.close()
    if world > 1:
        dist.destroy_process_group()


def run_sustained(step, alg, steps, index, torch, peak):
    """The step repeated for about half a second and longer, timed in chunks of 25 launches with CUDA events, the
    SM clock read through NVML once per chunk: throughput binned by the clock the GPU settled at.  On a 1 kW part
    the power cap pulls the clock down after some tens of milliseconds of this kernel; nothing is set or reset
    here, the clocks are only read."""
    chunk = 25
    n = max(steps // chunk, 8)
    try:
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(index)
    except Exception:
        return None
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    clocks, power = [], []
    ev[0].record()
    for c in range(n):
        for _ in range(chunk):
            step()
        ev[c + 1].record()
        if c >= 4:
            ev[c - 3].synchronize()          # a short queue, so that the sample belongs to the chunks around it
            clocks.append(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
            power.append(pynvml.nvmlDeviceGetPowerUsage(h) / 1000.0)
    torch.cuda.synchronize()
    ms = [ev[c].elapsed_time(ev[c + 1]) / chunk for c in range(n)]
    bins = {}
    for c, mhz in enumerate(clocks):
        bins.setdefault(int(round(mhz / 50.0) * 50), []).append(ms[c + 1])
    out = {str(k): {"chunks": len(v), "frac_hbm_measured": alg / (sum(v) / len(v) * 1e-3) / 1e9 / peak,
                    "ms_times_mhz": sum(v) / len(v) * k} for k, v in sorted(bins.items())}
    lowest = min(bins) if bins else None
    return {"steps": n * chunk, "seconds": sum(ms) * chunk * 1e-3, "chunk_launches": chunk, "by_sm_mhz": out,
            "lowest_sm_mhz": lowest, "frac_at_lowest_clock": out[str(lowest)]["frac_hbm_measured"] if bins else None,
            "first_chunk_frac": alg / (ms[0] * 1e-3) / 1e9 / peak, "last_chunk_frac": alg / (ms[-1] * 1e-3) / 1e9 / peak,
            "power_w_max": max(power) if power else None}


def run_host_cost():
    """Host microseconds per C-ABI call on the small tensor, measured by the C program of the package (no Python in
    the timed loop); None if it cannot be built or run."""
    import subprocess
    try:
        from paper_2603_02883_b200 import build as _b
        exe = _b.build_hostcost()
        r = subprocess.run([exe, "200", "20"], capture_output=True, text=True, timeout=120)
        if r.returncode != 0:
            return {"error": (r.stderr or r.stdout).strip()[-200:]}
        return json.loads(r.stdout.strip().splitlines()[-1])
    except Exception as e:   # no gcc / no CUDA headers on this machine
        return {"error": str(e)[-200:]}


def quality_report(ops, torch, fb4):
    """What the plain step produced: mean squared error of the decoded tensor (fp64 accumulation,
    over the first 8192 tokens) and how often each dialect was chosen."""
    q, x, T, C, B = ops.q, ops.x, ops.T, ops.C, ops.B
    codes, meta = ops.buf("codes", (T, C // 2), torch.uint8), ops.buf("meta", (T, C // B), torch.int16)
    fb4.fb4_quantize(q.ctx, x, T, C, C, codes, meta)
    n = min(T, 8192)
    dec = torch.empty((n, C), dtype=torch.float32, device="cuda")
    fb4.fb4_dequantize(q.ctx, codes[:n], meta[:n], n, C, None, 0, None, None, dec, 0)
    xs = x[:n].double()
    mse = float(((dec.double() - xs) ** 2).mean())
    power = float((xs ** 2).mean())
    did = (meta.to(torch.int32) >> 8) & 31
    hist = torch.bincount(did.flatten(), minlength=32).double()
    return {"mse_first_8192_tokens": mse, "signal_power": power, "sqnr_db": 10 * float(np.log10(power / mse)),
            "dialect_share": [round(float(v), 5) for v in (hist / hist.sum()).tolist()]}


def run_variants(ops, args, torch, fb4, synth, peak):
    """The other library paths on the same device, each timed like the headline step."""
    q, w, B = ops.q, ops.w, 32
    res = {}
    steps, warm = max(3, min(args.steps // 2, 20)), 5
    for name in OP_NAMES:
        if name == args.op:
            continue
        fn, alg = ops.get(name)
        total, per = time_steps(fn, steps, warm, torch)
        ms = total / steps
        res[name] = {"ms": ms, "GB/s": alg / (ms * 1e-3) / 1e9, "frac_hbm_measured": alg / (ms * 1e-3) / 1e9 / peak,
                     "kernel_variant": ("fast" if name.startswith("plain_") and name != "plain_f32" and name != "plain_block16" else q.last_variant) if name in ("plain", "plain_block16", "plain_every_element_a_group", "plain_all_dialects_scored", "plain_f32", "affine_plus_quantize", "layernorm_plus_quantize", "seda", "decomposed", "decomposed_given_set",
                                                                         "decomposed_seda", "quantize_mxfp8_tiled_scales",
                                                                         "quantize_mxfp8_decomposed_seda", "affine_plus_quantize_mxfp8")
                     else "decode"}
        if name == "dequantize_f32_decomposed":
            ops.drop("out32")
        if name == "plain_f32":
            ops.drop("x32")
    ops.drop("out16")
    if w.name != "c2":
        w2 = synth.workloads()["c2"]
        x2 = torch.from_numpy(synth.activation(w2).view(np.int16)).cuda().view(torch.bfloat16)
        c2 = torch.empty((w2.T, w2.C // 2), dtype=torch.uint8, device="cuda")
        m2 = torch.empty((w2.T, w2.C // B), dtype=torch.int16, device="cuda")
        # 258 MB per step is not far above the 126 MB L2: flush with a 512 MB write between steps
        flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
        evs = []
        for i in range(warm + steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fb4.fb4_quantize(q.ctx, x2, w2.T, w2.C, w2.C, c2, m2)
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        ms = float(np.mean([a.elapsed_time(b) for a, b in evs[warm:]]))
        alg = algorithmic_bytes(w2.T, w2.C)
        # offline weight quantizer on the same tensor, and how often the online (LUT, two-stage)
        # choice differs from the exhaustive exact-error choice (the paper's Table 2 comparison)
        cw2, mw2 = torch.empty_like(c2), torch.empty_like(m2)
        tot, _ = time_steps(lambda: fb4.fb4_quantize_weights(q.ctx, x2, w2.T, w2.C, w2.C, cw2, mw2), 3, 1, torch)
        dis = float(((m2.view(torch.int16).to(torch.int32) >> 8) != (mw2.view(torch.int16).to(torch.int32) >> 8))
                    .float().mean())
        o_a = torch.empty((w2.T, w2.C), dtype=torch.float32, device="cuda")
        fb4.fb4_dequantize(q.ctx, c2, m2, w2.T, w2.C, None, 0, None, None, o_a, 0)
        mse_lut = float(((o_a - x2.float()).double() ** 2).mean())
        fb4.fb4_dequantize(q.ctx, cw2, mw2, w2.T, w2.C, None, 0, None, None, o_a, 0)
        mse_exh = float(((o_a - x2.float()).double() ** 2).mean())
        del o_a
        res["c2_weights_exhaustive"] = {"ms": tot / 3, "Gelem/s": w2.T * w2.C / (tot / 3 * 1e-3) / 1e9,
                                        "dialect_disagreement_vs_online": dis,
                                        "mse_online_over_mse_exhaustive": mse_lut / mse_exh}
        # the small tensor (256 x 3072): launch-latency-bound; quantize + decode as a pair, launched
        # one by one and replayed from a CUDA graph of 20 pairs
        w1 = synth.workloads()["c1"]
        x1 = torch.from_numpy(synth.activation(w1).view(np.int16)).cuda().view(torch.bfloat16)
        c1 = torch.empty((w1.T, w1.C // 2), dtype=torch.uint8, device="cuda")
        m1 = torch.empty((w1.T, w1.C // B), dtype=torch.int16, device="cuda")
        o1 = torch.empty((w1.T, w1.C), dtype=torch.float32, device="cuda")

        def pair():
            fb4.fb4_quantize(q.ctx, x1, w1.T, w1.C, w1.C, c1, m1)
            fb4.fb4_dequantize(q.ctx, c1, m1, w1.T, w1.C, None, 0, None, None, o1, 0)

        tot, _ = time_steps(pair, 200, 20, torch)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            pair()
        torch.cuda.current_stream().wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for _ in range(20):
                pair()
        tot_g, _ = time_steps(graph.replay, 20, 3, torch)
        # salient-token selection, both readings, for the two sequence lengths of the workloads
        sel = {}
        for T_sel in (32760, 75600):
            sc_sel = torch.rand(T_sel, device="cuda", generator=torch.Generator(device="cuda").manual_seed(T_sel))
            out_sel = torch.empty(T_sel, dtype=torch.int32, device="cuda")
            t_tile, _ = time_steps(lambda: fb4.fb4_select_salient(q.ctx, sc_sel, T_sel, 20, out_sel), 20, 3, torch)
            t_topk, _ = time_steps(lambda: fb4.fb4_select_salient_topk(q.ctx, sc_sel, T_sel, T_sel // 20, out_sel), 20, 3,
                                   torch)
            sel[f"T={T_sel}"] = {"one_per_tile_of_20_us": t_tile / 20 * 1e3, "global_top_5_percent_us": t_topk / 20 * 1e3}
        res["salient_selection_launched_from_a_stream"] = sel
        res["c1_256x3072_quantize_plus_decode"] = {"us_per_pair_launched_one_by_one": tot / 200 * 1e3,
                                                   "us_per_pair_in_a_cuda_graph": tot_g / (20 * 20) * 1e3}
        # context for that size: a library copy that moves the same number of bytes (half read, half
        # written), timed the same way with the same flush
        half = torch.empty(int(alg) // 4, dtype=torch.int16, device="cuda")
        half2 = torch.empty_like(half)
        cevs = []
        for i in range(warm + steps):
            flush.zero_()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            half2.copy_(half)
            b.record()
            cevs.append((a, b))
        torch.cuda.synchronize()
        copy_ms = float(np.mean([a.elapsed_time(b) for a, b in cevs[warm:]]))
        res["c2_plain_32760x3072_l2_flushed"] = {"ms": ms, "GB/s": alg / (ms * 1e-3) / 1e9,
                                                 "frac_hbm_measured": alg / (ms * 1e-3) / 1e9 / peak,
                                                 "kernel_variant": q.last_variant,
                                                 "library_copy_of_the_same_bytes_ms": copy_ms,
                                                 "frac_of_that_copy": copy_ms / ms}
    return res


def run_e2e(q, bits, w, args, torch, fb4, barrier):
    """Same step through fb4_quantize_host: pinned host input -> device -> pinned host codes/meta,
    copies inside the timed region."""
    T, C, B = w.T, w.C, 32
    xh = torch.from_numpy(bits.view(np.int16)).pin_memory()
    ch = torch.empty((T, C // 2), dtype=torch.uint8).pin_memory()
    mh = torch.empty((T, C // B), dtype=torch.int16).pin_memory()
    dx = torch.empty((T, C), dtype=torch.int16, device="cuda")
    dc = torch.empty((T, C // 2), dtype=torch.uint8, device="cuda")
    dm = torch.empty((T, C // B), dtype=torch.int16, device="cuda")
    steps = max(2, min(args.steps, 5))
    fb4.fb4_quantize_host(q.ctx, xh, T, C, dx, dc, dm, ch, mh)
    torch.cuda.synchronize()
    if barrier:
        barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        fb4.fb4_quantize_host(q.ctx, xh, T, C, dx, dc, dm, ch, mh)
    torch.cuda.synchronize()
    dt = (time.perf_counter() - t0) / steps
    return {"value": None, "unit": UNIT, "h2d_bytes_per_step": T * C * 2,
            "d2h_bytes_per_step": T * C // 2 + T * (C // B) * 2, "seconds_per_step": dt, "steps": steps,
            "api": "fb4_quantize_host (pinned host buffers, chunked copies pipelined with the kernel)"}


def run_cpu_baseline(w, synth):
    from oracle import fb4_oracle as orc
    rows = min(w.T, 16384)
    bits = synth.activation_rows(w, 0, rows)
    fbk = synth.STANDIN_FORMATBOOK
    orc.quantize(bits[:256], fbk)
    reps, t0 = 0, time.perf_counter()
    while True:
        orc.quantize(bits, fbk)
        reps += 1
        if time.perf_counter() - t0 > 10.0 or reps >= 20:
            break
    dt = (time.perf_counter() - t0) / reps
    out = {"value": algorithmic_bytes(rows, w.C) / dt / 1e9, "unit": UNIT, "cores": os.cpu_count(),
           "kind": "oracle", "gelem_per_s": rows * w.C / dt / 1e9,
           "sample": f"first {rows} of {w.T} rows, {reps} passes, OpenMP over rows on all host cores"}
    # the same oracle on one core (its OpenMP runtime told to use one thread), on a 1024-row slab
    try:
        import ctypes
        gomp = ctypes.CDLL("libgomp.so.1")
        gomp.omp_get_max_threads.restype = ctypes.c_int
        before = gomp.omp_get_max_threads()
        gomp.omp_set_num_threads(1)
        try:
            slab = bits[:min(rows, 1024)]
            t0 = time.perf_counter()
            orc.quantize(slab, fbk)
            dt1 = time.perf_counter() - t0
        finally:
            gomp.omp_set_num_threads(before)
        out["one_core"] = {"value": algorithmic_bytes(slab.shape[0], w.C) / dt1 / 1e9, "unit": UNIT,
                           "gelem_per_s": slab.shape[0] * w.C / dt1 / 1e9,
                           "sample": f"first {slab.shape[0]} rows, one pass, one thread"}
    except OSError:
        pass
    return out


if __name__ == "__main__":
    main()
