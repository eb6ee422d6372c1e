"""Per-CTA timeline of the tile GEMM and attention launches of one denoise call at a large batch, from the kernels' own timer stamps.

    python -m paper_2608_03682_b200.trace_report [--batch 64] [--dtype bf16] [--first 100] [--last 107] [--option k=v ...]

For every launch index in [first, last) of the call (one layer of the batch-64 loop is seven launches: down of the
layer before, norm, q|k|v, attention, O, norm, gate/up) the option ``trace_all_from`` makes that launch, if it is a
tile GEMM or the tcgen05 attention kernel, stamp one slot per CTA (phyai_set_option "trace" / "trace_all_from", phyai_read_trace).  Printed per launch:
how long the CTAs spend in each phase, when the CTAs of each wave start and end, and the gap between two CTAs on the
same SM.  Stamps (ns, %globaltimer): 0 start, 1 barriers and tensor memory set up, 2 dependency resolved, 3 first
operands landed, 4 last MMA issued, 5 accumulator complete (persistent kernel: of its first tile), 6 epilogue's stores
issued, 7 SM id, 8 tensor memory released.  A traced call is a few per cent slower than an untraced one.
"""
import argparse

import numpy as np
import torch

from . import binding, synth

ATTN_PHASES = [("start -> dependency", 0, 1), ("dependency -> Q in tensor memory", 1, 2), ("-> S(0) issued", 2, 3),
               ("S(0) issued -> P V(0) issued", 3, 4), ("P V(0) issued -> all MMAs issued", 4, 5),
               ("last P V complete -> output stored", 6, 8), ("whole CTA", 0, 8)]
PHASES = [("start -> set up", 0, 1), ("set up -> dependency", 1, 2), ("dependency -> first operands", 2, 3),
          ("first operands -> last MMA issued", 3, 4), ("first accumulator complete -> stores issued", 5, 6),
          ("stores issued -> tensor memory released", 6, 8), ("whole CTA", 0, 8)]


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batch", type=int, default=64)
    ap.add_argument("--dtype", default="bf16")
    ap.add_argument("--first", type=int, default=100)
    ap.add_argument("--last", type=int, default=107)
    ap.add_argument("--option", action="append", default=[], help="key=value passed to phyai_set_option")
    a = ap.parse_args()
    B = a.batch
    cfg_id = 4 if a.dtype == "bf16" else 5
    cfg = synth.pi0_config(max_batch=B, dtype=a.dtype)
    ex = binding.Expert(cfg, binding.weights_to_device(synth.make_weights(cfg, cfg_id)))
    for kv_ in a.option:
        k, _, v = kv_.partition("=")
        ex.set_option(k, int(v))
    lens = [int(x) for x in synth.make_ragged_lengths(4, B, 600, 968)]
    kv_h, cu = synth.pack_prefix_kv([synth.make_prefix_kv(cfg, cfg_id, p, b) for b, p in enumerate(lens)])
    kv, cu_d = kv_h.cuda(), torch.from_numpy(cu).cuda()
    state = torch.stack([synth.make_state(cfg, cfg_id, b) for b in range(B)]).cuda()
    noise = torch.stack([synth.make_noise(cfg, cfg_id, b) for b in range(B)]).cuda()
    out = torch.empty_like(noise)
    ex.set_option("trace", 1)
    for base in range(a.first, a.last):
        ex.set_option("trace_all_from", base)
        for _ in range(2):
            ex.denoise_batched(kv, cu_d, state, noise, 10, out=out)
        torch.cuda.synchronize()
        tr = ex.read_trace().astype(np.int64)
        r = tr[tr[:, 0] != 0]
        if len(r) == 0:
            print(f"launch {base}: not a traced kernel")
            continue
        t0 = r[:, 0].min()
        if r[:, 10].max() == 1:   # the attention kernel: stamps 0 start, 1 dependency, 2 Q in tensor memory, 3 S(0) issued,
            # 4 P V(0) issued, 5 all MMAs issued, 6 last P V complete, 8 output stored, 9 key tiles
            print(f"launch {base}: attention, {len(r)} CTAs on {len(set(r[:, 7].tolist()))} SMs, span {(r[:, 8].max() - t0) / 1e3:.2f} us, "
                  f"key tiles per CTA {int(r[:, 9].min())}..{int(r[:, 9].max())}")
            for lab, i, j in ATTN_PHASES:
                v = (r[:, j] - r[:, i]) / 1e3
                print(f"   {lab:45s} min {v.min():7.2f}  p50 {np.median(v):7.2f}  p90 {np.percentile(v, 90):7.2f}  max {v.max():7.2f}")
            v = (r[:, 5] - r[:, 4]) / 1e3 / np.maximum(r[:, 9] - 1, 1)
            print(f"   {'per key tile after the first':45s} min {v.min():7.2f}  p50 {np.median(v):7.2f}  max {v.max():7.2f}")
            print(f"   sum of the CTAs' lives / SMs: {((r[:, 8] - r[:, 1]).clip(min=0).sum()) / 1e3 / 148:.2f} us")
            continue
        tiles = f", tiles per CTA {int(r[:, 9].min())}..{int(r[:, 9].max())}" if r[:, 9].max() > 0 else ""
        print(f"launch {base}: {len(r)} CTAs on {len(set(r[:, 7].tolist()))} SMs, span {(r[:, 8].max() - t0) / 1e3:.2f} us{tiles}")
        for lab, i, j in PHASES:
            v = (r[:, j] - r[:, i]) / 1e3
            print(f"   {lab:45s} min {v.min():7.2f}  p50 {np.median(v):7.2f}  p90 {np.percentile(v, 90):7.2f}  max {v.max():7.2f}")
        o = np.argsort(r[:, 0])
        print("   starts (sorted, every 37th CTA):", np.round((r[o, 0] - t0)[::37] / 1e3, 1))
        print("   ends   (same CTAs)             :", np.round((r[o, 8] - t0)[::37] / 1e3, 1))
        gaps = []
        for sm in set(r[:, 7].tolist()):
            rr = r[r[:, 7] == sm]
            rr = rr[np.argsort(rr[:, 0])]
            gaps += [(rr[i, 0] - rr[i - 1, 8]) / 1e3 for i in range(1, len(rr))]
        if gaps:
            print(f"   same SM, one CTA's end -> the next one's start: p50 {np.median(gaps):.2f} us, max {max(gaps):.2f} us")
    ex.close()


if __name__ == "__main__":
    main()
