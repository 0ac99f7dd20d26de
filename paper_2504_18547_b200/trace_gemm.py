"""Where the warp roles of the integer GEMM wait: a timeline of the four linear layers of one ViT-Base encoder layer.

    python -m paper_2504_18547_b200.trace_gemm [--batch 128] [--max-ctas N]

Builds the diagnostic library (-DVITINT_TRACE, a separate .so), runs one encoder-layer pass with the trace buffer
armed around each vitint_linear call and prints, for the first two CTAs and per role (TMA producer, MMA issuer, two
epilogue warps), the clock cycles spent blocked on each barrier and per-tile detail.  --max-ctas caps the persistent
grid (every tile is still computed, by fewer CTAs): comparing cycles per MMA of a CTA with 147 neighbours and with few
separates what an SM does to itself from what the chip's shared resources (L2, power) do to it.  Diagnostic only.
"""
from __future__ import annotations

import argparse
import ctypes
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent
if str(ROOT) not in sys.path:
    sys.path.insert(0, str(ROOT))

CTAS, ROLES, SLOTS = 4, 4, 4096
WAIT_EMPTY, GOT_EMPTY, WAIT_FULL, GOT_FULL, ISSUED, WAIT_ACC, GOT_ACC, TILE_DONE = 1, 2, 3, 4, 5, 6, 7, 8


def between(tags, clk, a, b):
    return sum(int(clk[i + 1] - clk[i]) for i in range(len(tags) - 1) if tags[i] == a and tags[i + 1] == b)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=128)
    ap.add_argument("--max-ctas", type=int, default=0)
    args = ap.parse_args()
    import torch

    import synth_inputs as si
    from paper_2504_18547_b200 import binding
    from paper_2504_18547_b200.build import build_trace_library
    binding._LIB_PATH = build_trace_library()
    from paper_2504_18547_b200 import encoder
    L = binding.lib()
    L.vitint_trace_set.argtypes = [ctypes.c_void_p]
    L.vitint_trace_max_ctas(int(args.max_ctas))
    cfg = si.VIT_BASE_LAYER.with_(batch=args.batch)
    prm = si.layer_parameters(cfg)
    dev = torch.device("cuda", 0)
    layer = encoder.EncoderLayer(cfg.batch, cfg.tokens, cfg.heads, cfg.mlp_dim, cfg.bits, prm, dev)
    x = torch.from_numpy(si.activations(cfg)).to(dev)
    out = torch.empty((cfg.rows, cfg.dim), dtype=torch.float32, device=dev)
    for _ in range(4):
        layer.forward(x, out)
    torch.cuda.synchronize()
    buf = torch.zeros(L.vitint_trace_words(), dtype=torch.int64, device=dev)
    traces = []
    plain = binding.vitint_linear

    def traced(*a, **k):
        torch.cuda.synchronize()
        buf.zero_()
        L.vitint_trace_set(buf.data_ptr())
        r = plain(*a, **k)
        torch.cuda.synchronize()
        L.vitint_trace_set(None)
        traces.append(buf.cpu().numpy().copy())
        return r
    encoder.B.vitint_linear = traced
    layer.forward(x, out)
    torch.cuda.synchronize()
    k_of = {"qkv": cfg.dim, "proj": cfg.dim, "fc1": cfg.dim, "fc2": cfg.mlp_dim}
    for name, t in zip(("qkv", "proj", "fc1", "fc2"), traces):
        t = t.reshape(CTAS, ROLES, SLOTS)
        print(f"== {name}" + (f" (grid capped at {args.max_ctas} CTAs)" if args.max_ctas else ""))
        for cta in range(2):
            rec = []
            for role in range(ROLES):
                n = int(t[cta, role, 0])
                r = t[cta, role, 1:1 + n]
                rec.append(((r & 255).astype(int), r >> 8))
            tags, clk = rec[0]
            print(f" cta{cta} TMA producer: span {int(clk[-1] - clk[0])} clk, blocked on a free stage {between(tags, clk, WAIT_EMPTY, GOT_EMPTY)}")
            tags, clk = rec[1]
            tiles = int((tags == ISSUED).sum())
            span, b_acc, b_ops = int(clk[-1] - clk[0]), between(tags, clk, WAIT_EMPTY, GOT_EMPTY), between(tags, clk, WAIT_FULL, GOT_FULL)
            mmas = tiles * (k_of[name] // 32)
            print(f" cta{cta} MMA issuer: span {span} clk over {tiles} tiles, blocked on an accumulator buffer "
                  f"{b_acc}, on operands {b_ops}; {mmas} MMAs, {span / max(mmas, 1):.0f} clk per MMA over the span, "
                  f"{(span - b_acc - b_ops) / max(mmas, 1):.0f} while issuing")
            for role in (2, 3):
                tags, clk = rec[role]
                work = [int(clk[i + 1] - clk[i]) for i in range(len(tags) - 1) if tags[i] == GOT_ACC and tags[i + 1] == TILE_DONE]
                print(f" cta{cta} epilogue warp ({'first' if role == 2 else 'last'}): span {int(clk[-1] - clk[0])}, group barrier "
                      f"{between(tags, clk, WAIT_ACC, WAIT_FULL)}, blocked on accumulators {between(tags, clk, WAIT_FULL, GOT_ACC)}, "
                      f"working {sum(work)} (per tile: {' '.join(map(str, work))})")
    print("device status", binding.vitint_device_status())


if __name__ == "__main__":
    main()
