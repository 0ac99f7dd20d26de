"""Benchmark of the integerized ViT-Base encoder layer (batch 128, 197 tokens, 4-bit W/A).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--bits 4]

One step = one pass of the whole hot path over one batch of synthetic activations:
LayerNorm+quantize -> QKV linear -> Q K^T -> scale+softmax+quantize -> P V -> projection ->
LayerNorm+quantize -> fc1 (GELU, requantize) -> fc2.  Prints ONE JSON line (rank 0).

value      effective TOPS (2 x true multiply-accumulates of the six integer contractions per
           second), inputs resident in HBM, whole job over all ranks (ranks hold disjoint images).
e2e        same metric through the same calls with every step's fp32 input copied from pinned host
           memory and its fp32 output copied back inside the timed region (copies of neighbouring
           steps overlap the kernels on separate streams).
roofline   the integer GEMM kernel: achieved TOPS over its launches inside the timed region
           (CUDA events around each call) against the int8 tensor peak.
cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

import synth_inputs as si  # noqa: E402

INT8_OVER_BF16 = 2.0          # nominal dense int8 : bf16 tensor throughput ratio on B200 (4.5 : 2.25 PFLOP/s)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
GEMM_DRAM_BYTES_PER_LAUNCH = 102.5e6   # ncu, ViT-Base layer, batch 128, 4-bit, byte codes: 410 MB over four launches
N_INPUT_BUFFERS = 4           # 4 x 77.5 MB of fp32 activations > 126 MB of L2


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", "100"], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        mhz = [float(r[0]) for r in self.rows if r and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) > 1 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for r in self.rows if len(r) >= 6 for n, v in zip(names, r[2:6]) if v.lower() == "active"})
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(mhz)}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def max_over_ranks(value: float, world: int, device=None) -> float:
    """MAX all-reduce of a scalar (identity for a single process)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def layer_ops(cfg: si.BlockConfig, batch: int) -> int:
    return 2 * batch * si.mac_counts(cfg.tokens, cfg.dim, cfg.heads, 64, cfg.mlp_dim)["total"]


# ---------------------------------------------------------------------------
# reference arm: the CPU oracle
# ---------------------------------------------------------------------------

def run_reference(args, cfg):
    rank, _, world = dist_env()
    if rank != 0:
        return
    import oracle as vo
    from oracle import pipeline as vp
    prm = si.layer_parameters(cfg)
    sample = args.ref_images
    x = si.activations(cfg, batch=sample)
    for _ in range(args.warmup):
        vp.encoder_layer(x[:cfg.tokens], prm, 1, cfg.tokens, cfg.heads, cfg.bits)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        vp.encoder_layer(x, prm, sample, cfg.tokens, cfg.heads, cfg.bits)
    dt = (time.perf_counter() - t0) / args.steps
    tops = layer_ops(cfg, sample) / dt / 1e12
    line = {
        "impl": "reference", "metric": "integerized ViT-B block effective TOPS", "value": tops, "unit": "TOPS",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "images_per_s": sample / dt,
        "config": {"workload": cfg.name, "bits": cfg.bits, "batch": cfg.batch, "tokens": cfg.tokens, "dim": cfg.dim,
                   "heads": cfg.heads, "mlp_dim": cfg.mlp_dim, "l2": "n/a (CPU)"},
        "cpu_baseline": {"value": tops, "unit": "TOPS", "cores": vo.get_threads(), "kind": "oracle",
                         "sample": f"{sample} of {cfg.batch} images per step, whole encoder layer"},
        "e2e": {"value": tops, "unit": "TOPS", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ---------------------------------------------------------------------------
# our arm
# ---------------------------------------------------------------------------

def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    import paper_2504_18547_b200 as vt
    from paper_2504_18547_b200.encoder import GEMM_STAGES, EncoderLayer

    rank, local_rank, world = dist_env()
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=device)

    prm = si.layer_parameters(cfg)
    layer = EncoderLayer(cfg.batch, cfg.tokens, cfg.heads, cfg.mlp_dim, cfg.bits, prm, device,
                         fused_attention=not args.unfused_attention,
                         wide_activations=not args.packed_activations)
    STAGES = layer.stages
    gemm_stages = [s for s in STAGES if s in GEMM_STAGES]
    M, D = cfg.rows, cfg.dim
    # each rank owns a disjoint range of images (weak scaling, no exchange on the data path)
    first = rank * cfg.batch
    host_x = [torch.from_numpy(si.activations(cfg, batch=cfg.batch, first_image=first + i * cfg.batch * world)
                               ).pin_memory() for i in range(N_INPUT_BUFFERS)]
    xs = [h.to(device) for h in host_x]
    out = torch.empty((M, D), dtype=torch.float32, device=device)
    host_out = torch.empty((M, D), dtype=torch.float32).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        layer.forward(xs[i % N_INPUT_BUFFERS], out)
    barrier()
    if vt.vitint_device_status() != 0:
        raise RuntimeError("device-side timeout during warm-up")

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.25)

    # ---- device-resident timing: exactly K steps back to back ---------------------------
    # No event sits between two kernels here: each kernel is launched as a programmatic dependent of the
    # one before it, and a stream operation in between would put the plain launch gap back.
    barrier()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for i in range(args.steps):
        layer.forward(xs[i % N_INPUT_BUFFERS], out)
    t_end.record()
    barrier()
    ms_total = max_over_ranks(t_start.elapsed_time(t_end), world, device)
    clocks = sampler.stop() if rank == 0 else None

    # ---- per-stage breakdown: the same K steps again, with an event around every call ---
    ev_steps = []
    for i in range(args.steps):
        ev = []
        layer.forward(xs[i % N_INPUT_BUFFERS], out, events=ev)
        ev_steps.append(ev)
    torch.cuda.synchronize()

    stage_ms = {s: 0.0 for s in STAGES}
    for ev in ev_steps:
        for j, s in enumerate(STAGES):
            stage_ms[s] += ev[j].elapsed_time(ev[j + 1])
    stage_ms = {s: v / args.steps for s, v in stage_ms.items()}

    # ---- end to end: host -> device, step, device -> host, every step -----------------
    # Three streams, double-buffered device input and output: the copy of step i+1's input and the read-back
    # of step i-1's result overlap step i's kernels (every step still moves its own input and output).
    barrier()
    main = torch.cuda.current_stream()
    s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
    x_dev = [torch.empty_like(xs[0]) for _ in range(2)]
    out_dev = [torch.empty_like(out) for _ in range(2)]
    ev_in = [torch.cuda.Event() for _ in range(2)]       # input i landed
    ev_done = [torch.cuda.Event() for _ in range(2)]     # step i finished (its input buffer is free, its output ready)
    ev_read = [torch.cuda.Event() for _ in range(2)]     # output i read back (its output buffer is free)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    s_in.wait_stream(main)
    s_out.wait_stream(main)
    for i in range(args.steps):
        b = i & 1
        with torch.cuda.stream(s_in):
            if i >= 2:
                s_in.wait_event(ev_done[b])              # step i-2 no longer reads this input buffer
            x_dev[b].copy_(host_x[i % N_INPUT_BUFFERS], non_blocking=True)
            ev_in[b].record(s_in)
        main.wait_event(ev_in[b])
        if i >= 2:
            main.wait_event(ev_read[b])                  # step i-2's result has left this output buffer
        layer.forward(x_dev[b], out_dev[b])
        ev_done[b].record(main)
        with torch.cuda.stream(s_out):
            s_out.wait_event(ev_done[b])
            host_out.copy_(out_dev[b], non_blocking=True)
            ev_read[b].record(s_out)
    main.wait_stream(s_in)
    main.wait_stream(s_out)
    t1.record()
    barrier()
    ms_e2e = max_over_ranks(t0.elapsed_time(t1), world, device)
    if vt.vitint_device_status() != 0:
        raise RuntimeError("device-side timeout during the timed region")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    peaks_early = measured_peaks()

    peaks = peaks_early
    ops_step = layer_ops(cfg, cfg.batch)
    ms_step = ms_total / args.steps
    tops = world * ops_step / (ms_step * 1e-3) / 1e12
    e2e_tops = world * ops_step / (ms_e2e / args.steps * 1e-3) / 1e12

    sops = layer.stage_ops()
    gemm_ms = sum(stage_ms[s] for s in gemm_stages)
    gemm_ops = sum(sops[s] for s in gemm_stages)
    int8_peak = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12
    sbytes = layer.stage_bytes()
    kernels = {}
    for s in STAGES:
        k = {"ms": round(stage_ms[s], 4)}
        if s in sops:
            k["tops"] = round(sops[s] / (stage_ms[s] * 1e-3) / 1e12, 1)
            k["frac_int8_peak"] = round(k["tops"] / int8_peak, 4)
        if s in sbytes:
            k["gbs"] = round(sbytes[s] / (stage_ms[s] * 1e-3) / 1e9, 1)
            k["frac_hbm_peak"] = round(k["gbs"] / peaks["hbm_gbs"], 4)
        kernels[s] = k

    # ---- streaming kernels that the fused step does not launch, timed alone (HBM roofline) -------------
    standalone = {}
    if world == 1 and not args.no_standalone:
        def timed(fn, reps=10):
            for _ in range(3):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(reps):
                fn()
            b.record()
            torch.cuda.synchronize()
            return a.elapsed_time(b) / reps
        cb = 4 if cfg.bits == 3 else cfg.bits
        n_rows, T = cfg.batch * cfg.heads * cfg.tokens, cfg.tokens
        S = torch.randint(-300, 300, (n_rows, (T + 3) // 4 * 4), dtype=torch.int32, device=device)   # 242 MB > L2
        Pq = vt.Codes.empty(n_rows, T, cfg.bits, False, device)
        xq = vt.Codes.empty(M, D, cfg.bits, True, device)
        sm_bytes = n_rows * T * 4 + n_rows * ((T * cb + 7) // 8)
        q_bytes = M * D * 4 + M * D * cb // 8
        # the paper's own LayerNorm quantizer (Eq. 5 statistics + comparator), which the default step does not use
        lrefs, lflip = vt.fold_layernorm_references(prm["ln1_g"], prm["ln1_b"], prm["s_ln"], cfg.bits, True, D)
        lrefs, lflip = torch.from_numpy(lrefs).to(device), torch.from_numpy(lflip).to(device)
        lstats = torch.empty((M, 2), dtype=torch.float32, device=device)
        n_eps = float(np.float32(D * 1e-6))
        for name, fn, nbytes in (
                ("quantize", lambda: vt.vitint_quantize(xs[1], layer.s_ln, cfg.bits, True, out=xq), q_bytes),
                ("layernorm_compare_quant", lambda: vt.vitint_layernorm_compare_quantize(
                    xs[2], lrefs, lflip, n_eps, cfg.bits, True, out=xq, stats=lstats), q_bytes),
                ("softmax_quant", lambda: vt.vitint_softmax_quantize(S, T, layer.c, layer.s_p, cfg.bits, out=Pq), sm_bytes),
                ("softmax_shift_quant", lambda: vt.vitint_softmax_shift_quantize(S, T, layer.c * 1.4426950408889634,
                                                                                 layer.s_p, cfg.bits, out=Pq), sm_bytes)):
            ms = timed(fn)
            standalone[name] = {"ms": round(ms, 4), "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                                "frac_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks_early["hbm_gbs"], 4)}
        del S, Pq, xq
        # the attention module of the paper's power table at its own shapes (DeiT-S width, 198 tokens, 3-bit,
        # per-head comparator LayerNorm on Q and K, Eq. 4 softmax), batch 64
        from paper_2504_18547_b200.encoder import NormedAttention
        dcfg = si.DEIT_S_ATTENTION
        dprm, dqkn = si.layer_parameters(dcfg), si.qk_norm_parameters(dcfg)
        mod = NormedAttention(dcfg.batch, dcfg.tokens, dcfg.heads, dcfg.bits, dprm, dqkn, device)
        dx = torch.from_numpy(si.activations(dcfg)).to(device)
        ds_x = float(si.lsq_step(dx[:dcfg.tokens].cpu().numpy(), dcfg.bits, True))
        dxq = vt.vitint_quantize(dx, ds_x, dcfg.bits, True)
        ms = timed(lambda: mod.forward(dxq, ds_x))
        standalone["deit_s_attention_n198_b64"] = {"ms": round(ms, 4), "tops": round(mod.ops() / (ms * 1e-3) / 1e12, 1),
                                                   "images_per_s": round(dcfg.batch / (ms * 1e-3), 1), "launches": 10}
        del mod, dx, dxq
        # the same encoder layer with the paper's own quantizers throughout (Eq. 4 softmax with the division-free
        # comparator, Eq. 5 statistics with the comparator LayerNorm quantizer): unfused attention, 11 launches
        from paper_2504_18547_b200.encoder import EncoderLayer as _Layer
        plain = _Layer(cfg.batch, cfg.tokens, cfg.heads, cfg.mlp_dim, cfg.bits, prm, device, softmax="shift",
                       layernorm="compare")
        ms = timed(lambda: plain.forward(xs[0], out), reps=5)
        standalone["layer_with_comparator_quantizers"] = {"ms": round(ms, 4), "tops": round(ops_step / (ms * 1e-3) / 1e12, 1),
                                                          "images_per_s": round(cfg.batch / (ms * 1e-3), 1),
                                                          "launches": len(plain.stages) + 2}
        del plain
        # the whole DeiT-S-shaped model (patch embedding, 198 tokens, 12 layers, final LayerNorm, two heads), batch 128
        from paper_2504_18547_b200.encoder import DeitModel
        mcfg = si.DEIT_S_MODEL
        model = DeitModel(si.model_end_parameters(mcfg), [si.layer_parameters(mcfg, layer=l) for l in range(mcfg.layers)],
                          mcfg.batch, mcfg.tokens, mcfg.heads, mcfg.mlp_dim, mcfg.bits, device)
        mp = torch.from_numpy(si.patch_rows(mcfg, batch=8)).to(device).repeat(mcfg.batch // 8, 1)
        ms = timed(lambda: model.forward(mp), reps=5)
        standalone["deit_s_model_n198_b128"] = {"ms": round(ms, 4), "tops": round(model.ops() / (ms * 1e-3) / 1e12, 1),
                                                "images_per_s": round(mcfg.batch / (ms * 1e-3), 1),
                                                "launches": 2 + 8 * mcfg.layers + 4}
        del model, mp
        # the 12-layer ViT-Base encoder at batch 256 (the multi-layer configuration): whole forward, images/s
        from paper_2504_18547_b200.encoder import EncoderStack
        ecfg = si.VIT_BASE_ENCODER.with_(bits=cfg.bits)
        stack = EncoderStack([si.layer_parameters(ecfg, layer=l) for l in range(ecfg.layers)], ecfg.batch, ecfg.tokens,
                             ecfg.heads, ecfg.mlp_dim, ecfg.bits, device)
        ex = torch.cat([xs[0], xs[1]])                       # 256 images of synthetic patch embeddings ~ N(0,1)
        eout = torch.empty_like(ex)
        ms = timed(lambda: stack.forward(ex, eout), reps=5)
        standalone["vit_base_encoder12_b256"] = {"ms": round(ms, 4), "tops": round(stack.ops() / (ms * 1e-3) / 1e12, 1),
                                                 "images_per_s": round(ecfg.batch / (ms * 1e-3), 1),
                                                 "launches": 8 * ecfg.layers}
        del stack, ex, eout

    # ---- CPU oracle on a bounded sample (rank 0, single-GPU runs only) -----------------
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        import oracle as vo
        from oracle import pipeline as vp
        sample = args.ref_images
        xs_cpu = si.activations(cfg, batch=sample)
        reps, t0c = 0, time.perf_counter()
        while True:                                  # about ten seconds of CPU work, whole passes only
            vp.encoder_layer(xs_cpu, prm, sample, cfg.tokens, cfg.heads, cfg.bits)
            reps += 1
            dtc = time.perf_counter() - t0c
            if dtc >= 10.0 or reps >= 20:
                break
        cpu = {"value": reps * layer_ops(cfg, sample) / dtc / 1e12, "unit": "TOPS", "cores": vo.get_threads(),
               "kind": "oracle",
               "sample": f"{sample} of {cfg.batch} images, whole encoder layer, {reps} passes in {dtc:.1f} s"}

    # DRAM bytes per GEMM launch (dram__bytes of one ncu capture of this workload, averaged over the step's four
    # launches; see profiles/).  Only valid for the default workload in its default layout.
    default_layout = (cfg.name == "vit_base_layer_b128" and cfg.bits == 4 and cfg.batch == 128 and layer.fused_attention
                      and not args.packed_activations)
    traffic = GEMM_DRAM_BYTES_PER_LAUNCH if default_layout else None
    line = {
        "metric": "integerized ViT-B block effective TOPS", "value": tops, "unit": "TOPS", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "int8", "data": "synthetic",
        "images_per_s": world * cfg.batch / (ms_step * 1e-3),
        "config": {"workload": cfg.name, "bits": cfg.bits, "batch_per_gpu": cfg.batch, "tokens": cfg.tokens,
                   "dim": cfg.dim, "heads": cfg.heads, "mlp_dim": cfg.mlp_dim,
                   "attention": "fused" if layer.fused_attention else "unfused",
                   "activation_codes": "packed" if args.packed_activations else "one per byte between linear layers",
                   "l2": f"inputs rotate over {N_INPUT_BUFFERS} buffers of {M * D * 4 / 1e6:.1f} MB (> 126 MB L2)"},
        "clocks": clocks,
        "e2e": {"value": e2e_tops, "unit": "TOPS", "h2d_bytes_per_step": M * D * 4, "d2h_bytes_per_step": M * D * 4,
                "ms_per_step": ms_e2e / args.steps},
        "gpu_launches": len(STAGES) * args.steps,
        "roofline": {"bound": "tensor", "kernel": f"gemm_i8_kernel ({len(gemm_stages)} launches per step)", "achieved": achieved,
                     "peak": int8_peak, "unit": "TOPS", "frac": achieved / int8_peak, "traffic": traffic,
                     "timing": "CUDA events around every call, second pass over the same K steps (the timed K steps carry no events)",
                     "peak_source": f"{peaks['source']} sustained bf16 cuBLAS x {INT8_OVER_BF16:g} (nominal int8:bf16)",
                     "frac_of_nominal_4500": achieved / 4500.0},
        "kernels": kernels,
        "kernels_standalone": standalone,
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------
# sweep: integer linear over K, N, tokens and bits; streaming kernels at the same sizes
# ---------------------------------------------------------------------------

SWEEP_KN = (192, 384, 768, 1024, 3072, 4096)
SWEEP_TOKENS_BATCH = ((197, 256), (577, 64), (785, 32))


def run_sweep(args):
    """Times vitint_linear (requantizing epilogue) for every K, N of SWEEP_KN at M = tokens x batch, 4-bit codes
    stored one per byte and 8-bit codes, against the int8 tensor roofline, and the quantize and softmax kernels at
    the same token counts against the HBM roofline.  Prints ONE JSON line; operands are seeded and synthetic
    (uniform random codes, which is all the timing depends on)."""
    import torch

    import paper_2504_18547_b200 as vt

    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    peaks = measured_peaks()
    int8_peak = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
    gen = torch.Generator(device=device)
    gen.manual_seed(si.BASE_SEED)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)       # larger than L2

    def timed(fn, reps):
        for _ in range(3):
            fn()
        t = 0.0
        for _ in range(reps):
            flush.zero_()                                                   # L2 flushed between timed iterations
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            torch.cuda.synchronize()
            t += a.elapsed_time(b)
        return t / reps

    def codes(rows, cols, bits):
        qn, qp = si.code_range(bits, True)
        t = torch.randint(qn, qp + 1, (rows, cols), dtype=torch.int8, device=device, generator=gen)
        return vt.Codes(t.view(torch.uint8), rows, cols, bits, True, 8)

    sampler = ClockSampler(0)
    sampler.start()
    linear = []
    for tokens, batch in SWEEP_TOKENS_BATCH:
        M = tokens * batch
        for bits in (4, 8):
            for K in SWEEP_KN:
                x = codes(M, K, bits)
                for N in SWEEP_KN:
                    w = codes(N, K, bits)
                    alpha = torch.full((N,), 1.0 / (K ** 0.5 * 2.0 ** (bits - 1)), dtype=torch.float32, device=device)
                    beta = torch.zeros((N,), dtype=torch.float32, device=device)
                    epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=alpha, beta=beta, out_bits=bits, out_signed=True,
                                      out_container=8)
                    out = vt.Codes.empty(M, N, bits, True, device, container=8)
                    ms = timed(lambda: vt.vitint_linear(x, 1.0, w, None, None, epi, out=out), args.steps)
                    tops = 2.0 * M * N * K / (ms * 1e-3) / 1e12
                    linear.append({"tokens": tokens, "batch": batch, "bits": bits, "K": K, "N": N, "ms": round(ms, 4),
                                   "tops": round(tops, 1), "frac_int8_peak": round(tops / int8_peak, 4)})
                    del w, out
                del x
    streaming = []
    for tokens, batch in SWEEP_TOKENS_BATCH:
        M = tokens * batch
        for bits in (2, 4, 8):
            cb = bits
            xf = torch.randn((M, 768), dtype=torch.float32, device=device, generator=gen)
            xq = vt.Codes.empty(M, 768, bits, True, device)
            ms = timed(lambda: vt.vitint_quantize(xf, 0.25, bits, True, out=xq), args.steps)
            nbytes = M * 768 * 4 + M * 768 * cb // 8
            streaming.append({"kernel": "quantize", "rows": M, "cols": 768, "bits": bits, "ms": round(ms, 4),
                              "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                              "frac_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)})
            rows = min(batch, 32) * 12 * tokens                     # attention rows of up to 32 images, 12 heads
            S = torch.randint(-300, 300, (rows, (tokens + 3) // 4 * 4), dtype=torch.int32, device=device, generator=gen)
            Pq = vt.Codes.empty(rows, tokens, bits, False, device)
            nbytes = rows * tokens * 4 + rows * ((tokens * cb + 7) // 8)
            for name, fn in (("softmax_quantize", lambda: vt.vitint_softmax_quantize(S, tokens, 0.01, 0.02, bits, out=Pq)),
                             ("softmax_shift_quantize", lambda: vt.vitint_softmax_shift_quantize(S, tokens, 0.0144, 0.02, bits, out=Pq))):
                ms = timed(fn, args.steps)
                streaming.append({"kernel": name, "rows": rows, "cols": tokens, "bits": bits, "ms": round(ms, 4),
                                  "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                                  "frac_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)})
            del xf, xq, S, Pq
    clocks = sampler.stop()
    if vt.vitint_device_status() != 0:
        raise RuntimeError("device-side timeout during the sweep")
    best = max(linear, key=lambda r: r["tops"])
    print(json.dumps({"metric": "integerized linear sweep, effective TOPS", "value": best["tops"], "unit": "TOPS",
                      "n_gpus": 1, "steps": args.steps, "warmup": 3, "higher_is_better": True, "dtype": "int8",
                      "data": "synthetic", "config": {"workload": "linear_and_streaming_sweep", "K_N": list(SWEEP_KN),
                                                      "tokens_batch": [list(t) for t in SWEEP_TOKENS_BATCH],
                                                      "l2": "256 MB written between timed iterations"},
                      "peaks": {"int8_tops": int8_peak, "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"]},
                      "clocks": clocks, "best": best, "linear": linear, "streaming": streaming}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--bits", type=int, default=4, choices=[2, 3, 4])
    ap.add_argument("--batch", type=int, default=None, help="images per GPU (default: the configuration's 128)")
    ap.add_argument("--ref-images", type=int, default=None, help="images per step of the CPU oracle")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep", action="store_true",
                    help="time the integer linear over K, N, tokens and bits, and the streaming kernels (one JSON line)")
    ap.add_argument("--no-standalone", action="store_true",
                    help="skip the kernels and composed workloads that are timed alone after the step")
    ap.add_argument("--packed-activations", action="store_true",
                    help="keep every activation code matrix bit-packed (default: one code per byte where only a linear layer reads it)")
    ap.add_argument("--unfused-attention", action="store_true", help="run Q K^T, softmax and P V as separate kernels")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    cfg = si.VIT_BASE_LAYER.with_(bits=args.bits)
    if args.batch:
        cfg = cfg.with_(batch=args.batch, name=f"vit_base_layer_b{args.batch}")
    if args.ref_images is None:
        args.ref_images = 64 if args.impl == "ours" else 8
    args.ref_images = min(args.ref_images, cfg.batch)
    if args.sweep:
        if dist_env()[0] == 0:
            run_sweep(args)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
