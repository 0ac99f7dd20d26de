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
GEMM_DRAM_BYTES_PER_LAUNCH = 101.5e6   # ncu, ViT-Base layer, batch 128, 4-bit, byte codes: 405.9 MB (read + write) over four launches
N_INPUT_BUFFERS = 4           # 4 x 77.5 MB of fp32 activations > 126 MB of L2


def measured_peaks():
    p = ROOT / "MEASURED_PEAKS.json"
    if p.exists():
        d = json.loads(p.read_text())
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d} | {"source": "measured"}
    return dict(FALLBACK_PEAKS) | {"source": "fallback"}


class ClockSampler:
    """Samples the SM clock and the clock-event (throttle) reasons of one GPU while timed regions run.

    Readings come from NVML (the library nvidia-smi itself reads; read-only queries) every ~2 ms on a thread of
    this process, each with a host timestamp, so that a region only a few milliseconds long still gets samples
    taken INSIDE it: window(t0, t1) summarises the samples whose timestamps fall between two perf_counter()
    readings.  Without NVML it falls back to polling `nvidia-smi -lms 20`."""
    NAMES = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
    MASKS = (0x8, 0x40, 0x20, 0x4)      # NVML clock-event reason bits, in the order of NAMES
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int, pci_bus_id: str | None = None):
        self.index, self.pci, self.samples, self.source = index, pci_bus_id, [], None
        self._stop = threading.Event()
        self._thread = self._proc = None
        self.max_mhz = None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            try:
                h = pynvml.nvmlDeviceGetHandleByPciBusId(self.pci.encode()) if self.pci else None
            except Exception:
                h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
            reasons_fn = getattr(pynvml, "nvmlDeviceGetCurrentClocksEventReasons", None) or \
                pynvml.nvmlDeviceGetCurrentClocksThrottleReasons

            def read_once():
                try:
                    mhz = float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM))
                    mask = int(reasons_fn(h))
                    self.samples.append((time.perf_counter(), mhz, mask))
                except Exception:
                    pass
            self._read_once = read_once

            def poll():
                while not self._stop.is_set():
                    read_once()
                    time.sleep(0.001)
            self.source = "nvml"
            self._thread = threading.Thread(target=poll, daemon=True)
            self._thread.start()
            return
        except Exception:
            pass
        try:
            self._proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                           "-i", str(self.index), "-lms", "20"], stdout=subprocess.PIPE, text=True)

            def read():
                for line in self._proc.stdout:
                    c = [v.strip() for v in line.split(",")]
                    if len(c) >= 6 and c[0].replace(".", "").isdigit():
                        mask = sum(m for m, v in zip(self.MASKS, c[2:6]) if v.lower() == "active")
                        self.samples.append((time.perf_counter(), float(c[0]), mask))
                        if c[1].replace(".", "").isdigit():
                            self.max_mhz = float(c[1])
            self.source = "nvidia-smi"
            self._thread = threading.Thread(target=read, daemon=True)
            self._thread.start()
        except OSError:
            self.source = None

    def sample_now(self):
        """One reading taken by the calling thread (used right after a burst of launches has been enqueued, while the
        GPU is still working through it: a burst of a few milliseconds may otherwise fall between two polls)."""
        fn = getattr(self, "_read_once", None)
        if fn is not None:
            fn()

    def window(self, t0: float, t1: float) -> dict:
        """Median SM clock and the union of the reasons over the samples taken in [t0, t1]."""
        if self.source is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no clock source"], "samples": 0}
        sel = [x for x in list(self.samples) if t0 <= x[0] <= t1]
        reasons = sorted({n for _, _, mask in sel for n, m in zip(self.NAMES, self.MASKS) if mask & m})
        return {"sm_mhz": float(np.median([x[1] for x in sel])) if sel else None, "sm_max_mhz": self.max_mhz,
                "reasons": reasons, "samples": len(sel), "source": self.source}

    def stop(self):
        self._stop.set()
        if self._proc is not None:
            self._proc.terminate()


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

    pci = None
    try:
        pr = torch.cuda.get_device_properties(local_rank)
        pci = "%08x:%02x:%02x.0" % (pr.pci_domain_id, pr.pci_bus_id, pr.pci_device_id)
    except Exception:
        pass
    sampler = ClockSampler(local_rank, pci)
    if rank == 0:
        sampler.start()
        time.sleep(0.05)

    def timed_steps(n):
        """n steps back to back, timed with CUDA events on the launching stream, max over ranks; also returns
        the host-clock window of the region for the clock samples."""
        # No event sits between two kernels here: each kernel is launched as a programmatic dependent of the
        # one before it, and a stream operation in between would put the plain launch gap back.
        barrier()
        w0 = time.perf_counter()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for i in range(n):
            layer.forward(xs[i % N_INPUT_BUFFERS], out)
            if rank == 0 and (i + 1) % 8 == 0:
                sampler.sample_now()        # the launches run ahead of the GPU: this reading falls inside the region
        b.record()
        if rank == 0:
            sampler.sample_now()
        barrier()
        return max_over_ranks(a.elapsed_time(b), world, device), (w0, time.perf_counter())

    def stage_breakdown(n):
        """The same steps again with an event around every call: per-stage milliseconds."""
        ev_steps = []
        for i in range(n):
            ev = []
            layer.forward(xs[i % N_INPUT_BUFFERS], out, events=ev)
            ev_steps.append(ev)
        torch.cuda.synchronize()
        acc = {s: 0.0 for s in STAGES}
        for ev in ev_steps:
            for j, s in enumerate(STAGES):
                acc[s] += ev[j].elapsed_time(ev[j + 1])
        return {s: v / n for s, v in acc.items()}

    # ---- device-resident timing: exactly K steps back to back (a burst: a few milliseconds) ------------
    ms_total, win = timed_steps(args.steps)
    clocks = sampler.window(*win) if rank == 0 else None
    stage_ms = stage_breakdown(args.steps)

    # ---- sustained leg: the same step repeated for several seconds, clock sampled inside the loop -------
    sustained = None
    if args.sustain_seconds > 0:
        n_sus = max(args.steps, int(np.ceil(args.sustain_seconds * 1e3 / (ms_total / args.steps))))
        ms_sus, win_s = timed_steps(n_sus)
        stage_ms_sus = stage_breakdown(min(50, n_sus))          # taken right behind the loop, still at its clocks
        sustained = {"steps": n_sus, "seconds": ms_sus * 1e-3, "ms_per_step": ms_sus / n_sus,
                     "clocks": sampler.window(*win_s) if rank == 0 else None, "stage_ms": stage_ms_sus}
    if rank == 0:
        sampler.stop()

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
    # The K timed steps are a burst (milliseconds at the boost clock): their fractions are taken against the
    # burst figure of the measured bf16 peak; the sustained leg's against the sustained figure.
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
    int8_peak_sustained = peaks["bf16_tflops_sustained"] * INT8_OVER_BF16
    achieved = gemm_ops / (gemm_ms * 1e-3) / 1e12
    if sustained is not None:
        g_ms = sum(sustained["stage_ms"][s] for s in gemm_stages)
        sus_tops = world * ops_step / (sustained["ms_per_step"] * 1e-3) / 1e12
        sustained.update({"value": sus_tops, "unit": "TOPS",
                          "images_per_s": world * cfg.batch / (sustained["ms_per_step"] * 1e-3),
                          "gemm_achieved": gemm_ops / (g_ms * 1e-3) / 1e12, "gemm_peak": int8_peak_sustained,
                          "gemm_frac": gemm_ops / (g_ms * 1e-3) / 1e12 / int8_peak_sustained,
                          "stage_ms": {k: round(v, 4) for k, v in sustained["stage_ms"].items()}})
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
        sm_ws = torch.empty(vt.vitint_softmax_table_workspace_bytes(64 * (1 << (cb - 1)) ** 2), dtype=torch.uint8, device=device)
        vt.vitint_softmax_quantize_bounded(S, T, layer.c, layer.s_p, cfg.bits, 64 * (1 << (cb - 1)) ** 2, out=Pq, workspace=sm_ws)
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
                # (the exp table depends on the layer's steps only: built by the warm-up call below, then reused)
                ("softmax_quant_bounded", lambda: vt.vitint_softmax_quantize_bounded(
                    S, T, layer.c, layer.s_p, cfg.bits, 64 * (1 << (cb - 1)) ** 2, out=Pq, workspace=sm_ws,
                    table_ready=True), sm_bytes),
                ("softmax_shift_quant", lambda: vt.vitint_softmax_shift_quantize(S, T, layer.c * 1.4426950408889634,
                                                                                 layer.s_p, cfg.bits, out=Pq), sm_bytes)):
            ms = timed(fn)
            standalone[name] = {"ms": round(ms, 4), "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                                "frac_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks_early["hbm_gbs"], 4)}
        del S, Pq, xq, sm_ws
        # the attention module of the paper's power table at its own shapes (DeiT-S width, 198 tokens, 3-bit,
        # per-head comparator LayerNorm on Q and K, Eq. 4 softmax), batch 64
        from paper_2504_18547_b200.encoder import NormedAttention
        dcfg = si.DEIT_S_ATTENTION
        dprm, dqkn = si.layer_parameters(dcfg), si.qk_norm_parameters(dcfg)
        dx = torch.from_numpy(si.activations(dcfg)).to(device)
        ds_x = float(si.lsq_step(dx[:dcfg.tokens].cpu().numpy(), dcfg.bits, True))
        dxq = vt.vitint_quantize(dx, ds_x, dcfg.bits, True)
        # fused: the per-head LayerNorm + comparator quantizer runs in the QKV GEMM's epilogue and Eq. 4 inside the
        # attention core (2 launches), or with Q K^T, softmax and P V as three kernels (4 launches);
        # unfused: fp32 Q and K rows through memory and a LayerNorm kernel each (10 launches)
        for name, fused, core, launches in (("deit_s_attention_n198_b64", True, True, 2),
                                            ("deit_s_attention_n198_b64_three_attention_kernels", True, False, 4),
                                            ("deit_s_attention_n198_b64_unfused", False, False, 10)):
            mod = NormedAttention(dcfg.batch, dcfg.tokens, dcfg.heads, dcfg.bits, dprm, dqkn, device, fused=fused, fused_core=core)
            ms = timed(lambda: mod.forward(dxq, ds_x))
            standalone[name] = {"ms": round(ms, 4), "tops": round(mod.ops() / (ms * 1e-3) / 1e12, 1),
                                "images_per_s": round(dcfg.batch / (ms * 1e-3), 1), "launches": launches}
            if fused and core:
                ms_q = timed(lambda: vt.vitint_linear_qkv_norm(dxq, ds_x, mod.w_qkv, mod.s_w_all, mod.bias_all, mod.refs_all,
                                                               mod.flip_all, mod.n_eps, mod.alpha_v, mod.beta_v, mod.bits,
                                                               out=mod.qkv, stats=mod.stats_all))
                standalone["qkv_linear_with_head_layernorm_deit_s_b64"] = {
                    "ms": round(ms_q, 4), "tops": round(2 * 3 * mod.rows * mod.dim * mod.dim / (ms_q * 1e-3) / 1e12, 1)}
            del mod
        del dx, dxq
        # the same encoder layer with the paper's own quantizers throughout (Eq. 4 softmax with the division-free
        # comparator, Eq. 5 statistics with the comparator LayerNorm quantizer), attention fused (Eq. 4 inside the core)
        # and as three kernels
        from paper_2504_18547_b200.encoder import EncoderLayer as _Layer
        for name, fused in (("layer_with_comparator_quantizers", True), ("layer_with_comparator_quantizers_unfused_attention", False)):
            plain = _Layer(cfg.batch, cfg.tokens, cfg.heads, cfg.mlp_dim, cfg.bits, prm, device, softmax="shift",
                           layernorm="compare", fused_attention=fused)
            ms = timed(lambda: plain.forward(xs[0], out), reps=5)
            standalone[name] = {"ms": round(ms, 4), "tops": round(ops_step / (ms * 1e-3) / 1e12, 1),
                                "images_per_s": round(cfg.batch / (ms * 1e-3), 1), "launches": len(plain.stages) + 2}
            if fused:
                # the fused attention core alone on this layer's QKV codes: Eq. 4 inside against the exp table inside
                ws4 = torch.empty(vt.vitint_attention_core_shift_workspace_bytes(cfg.bits), dtype=torch.uint8, device=device)
                args4 = (plain.qkv, cfg.batch, cfg.heads, cfg.tokens, plain.s_q, plain.s_k, plain.s_p, cfg.bits, plain.alpha_o, None)
                vt.vitint_attention_core_shift(*args4, out=plain.O, workspace=ws4)
                ms_s = timed(lambda: vt.vitint_attention_core_shift(*args4, out=plain.O, workspace=ws4, table_ready=True))
                tab = vt.vitint_attention_exp_table(cfg.bits, plain.s_q, plain.s_k, device=device)
                ms_e = timed(lambda: vt.vitint_attention_core_prepared(*args4, out=plain.O, table=tab))
                att_ops = 2 * 2 * cfg.batch * cfg.heads * cfg.tokens * cfg.tokens * 64
                standalone["attention_core_eq4_softmax"] = {"ms": round(ms_s, 4), "tops": round(att_ops / (ms_s * 1e-3) / 1e12, 1)}
                standalone["attention_core_exp_softmax"] = {"ms": round(ms_e, 4), "tops": round(att_ops / (ms_e * 1e-3) / 1e12, 1)}
                del ws4, tab
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

    # ---- a library int8 GEMM in the same run, as context for the int8 ceiling (never on the product path) ----
    library_int8 = None
    if world == 1 and not args.no_standalone and hasattr(torch, "_int_mm"):
        try:
            n = 8192
            la = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=device)
            lb = torch.randint(-8, 8, (n, n), dtype=torch.int8, device=device).t()
            for _ in range(3):
                torch._int_mm(la, lb)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(10):
                torch._int_mm(la, lb)
            e1.record()
            torch.cuda.synchronize()
            library_int8 = 2.0 * n ** 3 * 10 / (e0.elapsed_time(e1) * 1e-3) / 1e12
            del la, lb
        except Exception:
            library_int8 = None

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
                     "peak_source": f"{peaks['source']} burst bf16 cuBLAS x {INT8_OVER_BF16:g} (nominal int8:bf16); the K steps are a burst",
                     "frac_of_nominal_4500": achieved / 4500.0,
                     "achieved_sustained": sustained["gemm_achieved"] if sustained else None,
                     "peak_sustained": int8_peak_sustained,
                     "frac_sustained": sustained["gemm_frac"] if sustained else None,
                     "library_int8_tops": library_int8,
                     "library_int8_note": "torch._int_mm 8192^3 in this run: context for the int8 ceiling, not on the product path"},
        "sustained": sustained,
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
SWEEP_BATCHES = {197: (1, 8, 64, 256), 577: (1, 8, 64), 785: (1, 8, 32)}
SWEEP_KN_THIN = ((192, 192), (768, 768), (768, 3072), (3072, 768), (4096, 4096))


def run_sweep(args):
    """The scaling study over K, N, tokens, batch and bit width.  ONE JSON line with five tables:
    linear          vitint_linear, requantizing epilogue, every K, N of SWEEP_KN at M = tokens x batch (the largest
                    batch per token count), 4-bit codes stored one per byte and 8-bit codes;
    linear_batch    the same call at batch 1 ... 256 on a thinned K, N grid;
    linear_formats  bit-packed 2-, 3- and 4-bit operands (activations packed, weights packed or widened once) and the
                    fp32 (dequantizing) epilogue;
    attention       the fused core (up to 256 tokens) and the unfused Q K^T -> softmax -> P V sequence (577 and 785
                    tokens), 12 heads, batch 1 ... 256;
    streaming       quantize and the two softmax kernels against the HBM roofline.
    GEMM-shaped points are given against the int8 tensor roofline.  Every point is timed alone with the L2 flushed
    before each timed call (a burst), so the tensor peak is the burst figure.  Operands are seeded and synthetic
    (uniform random codes, which is all the timing depends on)."""
    import torch

    import paper_2504_18547_b200 as vt

    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    peaks = measured_peaks()
    int8_peak = peaks["bf16_tflops"] * INT8_OVER_BF16
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

    def codes(rows, cols, bits, signed=True, container=8):
        """Random codes of the declared range, one per byte (container 8) or bit-packed."""
        qn, qp = si.code_range(bits, signed)
        t = torch.randint(qn, qp + 1, (rows, cols), dtype=torch.int8, device=device, generator=gen)
        if container == 8:
            return vt.Codes(t.view(torch.uint8), rows, cols, bits, signed, 8)
        c = 4 if bits == 3 else bits
        per = 8 // c
        v = (t.to(torch.int32) & ((1 << c) - 1)).view(rows, cols // per, per)
        sh = torch.arange(per, device=device, dtype=torch.int32) * c
        return vt.Codes((v << sh).sum(dim=2).to(torch.uint8).contiguous(), rows, cols, bits, signed, 0)

    def requant_epi(N, K, bits, container=8):
        alpha = torch.full((N,), 1.0 / (K ** 0.5 * 2.0 ** (bits - 1)), dtype=torch.float32, device=device)
        beta = torch.zeros((N,), dtype=torch.float32, device=device)
        return vt.Epilogue(mode=vt.EPI_REQUANT, alpha=alpha, beta=beta, out_bits=bits, out_signed=True,
                           out_container=container)

    def lin_point(M, K, N, bits, x, w, epi, out, **tags):
        ms = timed(lambda: vt.vitint_linear(x, 1.0, w, epi_args.get("w_step"), epi_args.get("bias"), epi, out=out), args.steps)
        tops = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        return dict(tags, bits=bits, K=K, N=N, M=M, ms=round(ms, 4), tops=round(tops, 1),
                    frac_int8_peak=round(tops / int8_peak, 4))

    epi_args = {}
    sampler = ClockSampler(0)
    sampler.start()
    w_start = time.perf_counter()
    linear = []
    for tokens, batch in SWEEP_TOKENS_BATCH:
        M = tokens * batch
        for bits in (4, 8):
            for K in SWEEP_KN:
                x = codes(M, K, bits)
                for N in SWEEP_KN:
                    w = codes(N, K, bits)
                    out = vt.Codes.empty(M, N, bits, True, device, container=8)
                    linear.append(lin_point(M, K, N, bits, x, w, requant_epi(N, K, bits), out, tokens=tokens, batch=batch))
                    del w, out
                del x
    linear_batch = []
    for tokens, batches in SWEEP_BATCHES.items():
        for batch in batches:
            M = tokens * batch
            for K, N in SWEEP_KN_THIN:
                x, w = codes(M, K, 4), codes(N, K, 4)
                out = vt.Codes.empty(M, N, 4, True, device, container=8)
                linear_batch.append(lin_point(M, K, N, 4, x, w, requant_epi(N, K, 4), out, tokens=tokens, batch=batch))
                del x, w, out
    linear_formats = []
    M = 197 * 64
    for K, N in ((768, 768), (768, 3072), (3072, 768)):
        for bits in (2, 3, 4):
            xp = codes(M, K, bits, container=0)
            for wname, w in (("packed", codes(N, K, bits, container=0)), ("one per byte", codes(N, K, bits))):
                out = vt.Codes.empty(M, N, bits, True, device)
                linear_formats.append(lin_point(M, K, N, bits, xp, w, requant_epi(N, K, bits, 0), out, activations="packed",
                                                weights=wname, epilogue="requantize, packed output"))
                del out
            del xp
        # fp32 epilogue (scale, bias, no residual) on codes stored one per byte
        x, w = codes(M, K, 4), codes(N, K, 4)
        epi_args = {"w_step": torch.full((N,), 0.01, dtype=torch.float32, device=device),
                    "bias": torch.zeros((N,), dtype=torch.float32, device=device)}
        outf = torch.empty((M, N), dtype=torch.float32, device=device)
        linear_formats.append(lin_point(M, K, N, 4, x, w, vt.Epilogue(mode=vt.EPI_DEQUANT_F32), outf, activations="one per byte",
                                        weights="one per byte", epilogue="fp32 (scale + bias)"))
        epi_args = {}
        del x, w, outf
    attention = []
    heads, D = 12, 768
    for tokens, batches in SWEEP_BATCHES.items():
        for batch in batches:
            M = tokens * batch
            ops = 4.0 * batch * heads * tokens * tokens * 64
            for bits in ((4, 2) if tokens <= 256 else (4,)):
                qmax = 1 << (bits - 1)
                s_qk = float(np.float32((3.0 / (qmax * qmax)) ** 0.5))
                s_p = float(np.float32(2.0 / (tokens * (2 ** bits - 1) ** 0.5)))
                alpha = torch.full((D,), 0.01, dtype=torch.float32, device=device)
                # the fused core: one pipeline pair per CTA up to 256 tokens, the chunked two-pass kernel beyond
                qkv = codes(M, 3 * D, bits)
                o = vt.Codes.empty(M, D, bits, True, device, container=8)
                table = vt.vitint_attention_exp_table(bits, s_qk, s_qk, device=device)
                ms = timed(lambda: vt.vitint_attention_core_prepared(qkv, batch, heads, tokens, s_qk, s_qk, s_p, bits,
                                                                     alpha, None, out=o, table=table), args.steps)
                attention.append({"path": "fused core" if tokens <= 256 else "fused core, keys in chunks (two passes)",
                                  "tokens": tokens, "batch": batch, "bits": bits,
                                  "ms": round(ms, 4), "tops": round(ops / (ms * 1e-3) / 1e12, 1)})
                del qkv, o
                if tokens > 256:
                    qkv = codes(M, 3 * D, bits, container=0)
                    sl = [vt.Slabs.of_qkv(qkv, tokens, D, i) for i in range(3)]
                    ld_s = (tokens + 3) // 4 * 4
                    S = torch.empty((batch * heads * tokens, ld_s), dtype=torch.int32, device=device)
                    P = vt.Codes.empty(batch * heads * tokens, tokens, bits, False, device)
                    o = vt.Codes.empty(M, D, bits, True, device)
                    epi = vt.Epilogue(mode=vt.EPI_REQUANT, alpha=alpha, out_bits=bits, out_signed=True)
                    c = float(np.float32(s_qk * s_qk / 8.0))
                    parts = {"qk": lambda: vt.vitint_qk(sl[0], sl[1], batch, heads, tokens, out=S, ld_s=ld_s),
                             "softmax_quantize": lambda: vt.vitint_softmax_quantize(S, tokens, c, s_p, bits, out=P),
                             "pv": lambda: vt.vitint_pv(P, sl[2], batch, heads, tokens, s_p, 0.1, epi, out=o)}
                    pm = {k: round(timed(f, args.steps), 4) for k, f in parts.items()}
                    ms = timed(lambda: [f() for f in parts.values()], args.steps)
                    sm_bytes = S.shape[0] * tokens * 4 + S.shape[0] * ((tokens * (4 if bits == 3 else bits) + 7) // 8)
                    attention.append({"path": "unfused qk -> softmax -> pv", "tokens": tokens, "batch": batch, "bits": bits,
                                      "ms": round(ms, 4), "tops": round(ops / (ms * 1e-3) / 1e12, 1), "kernel_ms": pm,
                                      "softmax_gbs": round(sm_bytes / (pm["softmax_quantize"] * 1e-3) / 1e9, 1),
                                      "softmax_frac_hbm_peak": round(sm_bytes / (pm["softmax_quantize"] * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)})
                    del qkv, S, P, o
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
            kernels = [("softmax_quantize", lambda: vt.vitint_softmax_quantize(S, tokens, 0.01, 0.02, bits, out=Pq)),
                       ("softmax_shift_quantize", lambda: vt.vitint_softmax_shift_quantize(S, tokens, 0.0144, 0.02, bits, out=Pq))]
            if tokens <= 895:
                # the table-driven kernel for scores of declared range (here 4096, the bound of 4-bit Q and K codes);
                # its table is built by an untimed first call and reused
                ws = torch.empty(vt.vitint_softmax_table_workspace_bytes(4096), dtype=torch.uint8, device=device)
                vt.vitint_softmax_quantize_bounded(S, tokens, 0.01, 0.02, bits, 4096, out=Pq, workspace=ws)
                kernels.insert(1, ("softmax_quantize_bounded", lambda: vt.vitint_softmax_quantize_bounded(
                    S, tokens, 0.01, 0.02, bits, 4096, out=Pq, workspace=ws, table_ready=True)))
            for name, fn in kernels:
                ms = timed(fn, args.steps)
                streaming.append({"kernel": name, "rows": rows, "cols": tokens, "bits": bits, "ms": round(ms, 4),
                                  "gbs": round(nbytes / (ms * 1e-3) / 1e9, 1),
                                  "frac_hbm_peak": round(nbytes / (ms * 1e-3) / 1e9 / peaks["hbm_gbs"], 4)})
            del xf, xq, S, Pq
    clocks = sampler.window(w_start, time.perf_counter())
    sampler.stop()
    if vt.vitint_device_status() != 0:
        raise RuntimeError("device-side timeout during the sweep")
    best = max(linear, key=lambda r: r["tops"])
    print(json.dumps({"metric": "integerized linear sweep, effective TOPS", "value": best["tops"], "unit": "TOPS",
                      "n_gpus": 1, "steps": args.steps, "warmup": 3, "higher_is_better": True, "dtype": "int8",
                      "data": "synthetic", "config": {"workload": "linear_and_attention_sweep", "K_N": list(SWEEP_KN),
                                                      "tokens_batch": [list(t) for t in SWEEP_TOKENS_BATCH],
                                                      "batches": {str(k): list(v) for k, v in SWEEP_BATCHES.items()},
                                                      "l2": "256 MB written between timed iterations"},
                      "peaks": {"int8_tops": int8_peak, "hbm_gbs": peaks["hbm_gbs"], "source": peaks["source"],
                                "int8_note": "burst bf16 cuBLAS x 2 (nominal int8 : bf16)"},
                      "clocks": clocks, "best": best, "linear": linear, "linear_batch": linear_batch,
                      "linear_formats": linear_formats, "attention": attention, "streaming": streaming}))


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
    ap.add_argument("--sustain-seconds", type=float, default=3.0,
                    help="length of the sustained leg that follows the K timed steps (0 = skip it)")
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
    rank, _, world = dist_env()
    if args.impl == "ours" and not args.sweep and args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: start one rank per GPU of this node and let rank 0 print the line
        import socket
        sk = socket.socket()
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
        sk.close()
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(port), str(Path(__file__).resolve())] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.impl == "ours" and not args.sweep and world != args.gpus:
        raise SystemExit(f"bench.py: --gpus {args.gpus} but {world} rank(s) were started (WORLD_SIZE); "
                         "start it with one rank per GPU or let bench.py start them itself")
    if args.sweep:
        if dist_env()[0] == 0:
            run_sweep(args)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
