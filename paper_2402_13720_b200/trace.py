"""Timeline of the kernels of one verification forward, from stamps taken inside the kernels.

    python -m paper_2402_13720_b200.trace [--config C2] [--cache-len 4096] [--rows 37] [--which target|draft]

Builds libouro_trace.so (the library compiled with -DOURO_TRACE: selected threads of every CTA of the weight GEMM
and of the tcgen05 attention stamp the GPU's nanosecond timer at fixed points), runs a few forwards of the chosen
configuration and prints, per kernel of the last forward, when its CTAs reached each point, relative to the moment
the kernel's dependency wait returned (= the previous kernel had completed).  The regular library is not touched.
"""
from __future__ import annotations

import argparse
import ctypes as C
import os
import sys

import numpy as np


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", default="C2")
    ap.add_argument("--cache-len", type=int, default=4096)
    ap.add_argument("--rows", type=int, default=37, help="block rows (1 = plain decoding step)")
    ap.add_argument("--which", default="target", choices=["target", "draft"])
    ap.add_argument("--layers", type=int, default=0, help="cut the model to this many layers (0: as configured)")
    args = ap.parse_args()
    from . import build
    os.environ["OURO_LIB"] = build.build(trace=True)
    import dataclasses
    import torch
    from . import binding, synth

    T, D, P, _ = synth.config(args.config)
    M = T if args.which == "target" else D
    if args.layers:
        M = dataclasses.replace(M, n_layers=args.layers)
    M = dataclasses.replace(M, max_seq=max(M.max_seq, args.cache_len + 160))
    w = synth.model_weights(M, 0, device="cuda:0")
    eng = binding.Engine(M, w, P)
    k, v = synth.kv_fill(M, 1, args.cache_len, device="cuda:0")
    eng.tm.k_cache.copy_(k)
    eng.tm.v_cache.copy_(v)
    tokens = np.arange(args.rows, dtype=np.int32) % M.vocab
    if args.rows == P.block_max:      # the candidate block itself: K phrases that start with the draft's last token
        grams = np.array([[3] + [(7 * j + i) % M.vocab for i in range(P.S)] for j in range(P.K)], dtype=np.int32)
        eng.phrase_update(grams)
    for _ in range(5):
        eng.set_state(args.cache_len, 17)
        if args.rows == P.block_max:
            eng.assemble_candidates(draft=[5, 6, 7, 3][-P.gamma:] if P.gamma <= 4 else list(range(P.gamma - 1)) + [3])
        else:
            eng.assemble_causal(binding.OURO_TARGET, tokens)
        eng.verify_forward()
    torch.cuda.synchronize()
    lib = binding.lib()
    g = (C.c_ulonglong * (8 * 160 * 16))()
    a = (C.c_ulonglong * (512 * 8))()
    assert lib.ouro_trace_read_gemm(g) == 0 and lib.ouro_trace_read_attn(a) == 0
    g = np.array(g[:], dtype=np.int64).reshape(8, 160, 16)
    a = np.array(a[:], dtype=np.int64).reshape(512, 8)
    if not (a[:, 0] > 0).any():                  # head dim 64: the mma.sync attention kernel keeps a timeline of its own
        assert lib.ouro_trace_read_attn_tc(a.ctypes.data_as(C.POINTER(C.c_ulonglong))) == 0

    def stats(x):
        return "min %6.1f  med %6.1f  max %6.1f" % (x.min(), np.median(x), x.max()) if len(x) else "-"

    names = ["q,k,v", "o-proj", "gate,up", "down", "LM head"]
    points = [(0, "CTA entry"), (8, "last weight load issued"), (2, "first stage full"), (3, "last MMA issued"),
              (4, "last accumulator complete"), (5, "whole tiles done / fix-up begins"), (6, "partials of the others there"),
              (9, "  group 0: past the wait + fence"), (12, "  group 0: first batch added up"), (10, "  group 0: its tokens finished"), (11, "  group 0: tile re-armed"),
              (7, "fix-up done")]
    spans = []
    for kind in range(5):
        t = g[kind]
        live = t[:, 1] > 0                       # stamped by every GEMM of a chained launch (slot 0: by its first only)
        if not live.any():
            continue
        t = t[live]
        t0 = t[:, 1].min()
        print(f"{names[kind]}  ({live.sum()} CTAs; us relative to the end of the dependency wait)")
        for col, nm in points:
            x = t[:, col][t[:, col] > 0]
            print("   %-34s %s" % (nm, stats((x - t0) / 1e3)))
        spans.append((names[kind], t0, max(t[:, 7].max(), t[:, 5].max())))
    live = a[:, 0] > 0
    if live.any():
        t = a[live]
        t0 = t[:, 2].min()
        print(f"attention  ({live.sum()} CTAs)")
        for col, nm in [(0, "CTA entry"), (1, "set-up done, waiting"), (2, "dependency wait over"), (3, "first scores"), (6, "(head dim 64) second chunk begins"), (7, "(head dim 64) third chunk begins"),
                        (4, "last pass accumulated"), (5, "CTA done")]:
            x = t[:, col][t[:, col] > 0]
            print("   %-34s %s" % (nm, stats((x - t0) / 1e3)))
        spans.append(("attention", t0, t[:, 5].max()))
    spans.sort(key=lambda s: s[1])
    print("in launch order: kernel, dependency wait over at (us), last CTA done at (us), length")
    base = spans[0][1]
    for nm, t0, t1 in spans:
        print("   %-10s %8.1f %8.1f %8.1f" % (nm, (t0 - base) / 1e3, (t1 - base) / 1e3, (t1 - t0) / 1e3))
    eng.close()


if __name__ == "__main__":
    sys.exit(main())
