"""Benchmark of the Ouroboros verification step on B200.

A step is one pass of the whole hot path over one synthetic batch: phrase lookup, candidate packing, one
target forward under the candidate mask (embedding, decoder layers, LM head, argmax), greedy acceptance,
KV compaction and phrase harvest.  Workload: one 7B-shaped decoder layer (d 4096, 32 heads, FFN 11008,
vocabulary 32000, bf16) on a 4096-token KV cache with a 37-row query block (1 + 4 draft tokens + 4 phrases
x 8 tokens).  The metric is the verify-step HBM throughput: algorithmic bytes of the step / step time.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--cache-len L]

N > 1 runs N independent replicas (one process per GPU under torchrun); the decoding stream of one query is
strictly sequential, so there is no data-path collective.  `--impl reference` times the CPU oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
GEMM_PROFILE = os.path.join(ROOT, "profiles", "gemm_tc_kernel_verify_step_c2.md")


def kernel_rev():
    """Hash of the device side of csrc/gemm_tc.cu: everything above its host-side part."""
    import hashlib
    with open(os.path.join(ROOT, "paper_2402_13720_b200", "csrc", "gemm_tc.cu"), "rb") as f:
        src = f.read()
    cut = src.find(b"host side")
    return hashlib.sha256(src[:cut] if cut > 0 else src).hexdigest()[:16]


def profiled_traffic():
    """DRAM bytes (read + write) per gemm_tc_kernel launch from the ncu capture summarised in profiles/: the summary
    carries a line `traffic_bytes_per_launch: <number> kernel_rev: <hash>`; the figure counts only while the kernel's
    device code still has that hash."""
    import re
    try:
        m = re.search(r"traffic_bytes_per_launch:\s*([0-9.e+]+)\s+kernel_rev:\s*([0-9a-f]+)", open(GEMM_PROFILE).read())
    except OSError:
        return None
    return float(m.group(1)) if m and m.group(2) == kernel_rev() else None

from paper_2402_13720_b200 import synth  # noqa: E402

METRIC, UNIT = "verify_step_hbm_throughput", "GB/s"
SEED = 0
PENDING = 17
PROF_CLASSES = ("qkv", "attention", "wo", "gateup", "down", "head")     # "gemm": every launch of the weight-streaming kernel


# ------------------------------------------------------------------------------ workload

def algorithmic_bytes(m: synth.ModelDesc, B: int, L: int) -> dict:
    """Bytes one verification step must move: every weight once, the visible KV cache once, the block's K/V
    written once, B embedding rows; activations (a few hundred KB, L2 resident) are not counted."""
    e = 2 if m.dtype == "bf16" else 4
    layer_w = m.layer_weight_elems() * e + 2 * m.d_model * e
    kv_read = 2 * L * m.d_kv * e
    kv_write = 2 * B * m.d_kv * e
    per_class = {
        "qkv": (m.d_q + 2 * m.d_kv) * m.d_model * e,
        "attention": kv_read + 2 * B * m.d_kv * e,
        "wo": m.d_model * m.d_q * e,
        "gateup": 2 * m.d_ffn * m.d_model * e,
        "down": m.d_ffn * m.d_model * e,
        "head": m.vocab * m.d_model * e,
    }
    total = m.n_layers * (layer_w + kv_read + kv_write) + m.vocab * m.d_model * e + m.d_model * e + B * m.d_model * e
    return dict(total=total, per_class=per_class, layers=m.n_layers)


def block_inputs(m: synth.ModelDesc, P: synth.DecodeParams):
    """Seeded draft tokens and K phrases that start with the draft's last token."""
    draft = np.array([synth.hash_u64(SEED, 70, i) % m.vocab for i in range(P.gamma)], dtype=np.int32)
    grams = np.array([[draft[-1]] + [synth.hash_u64(SEED, 71, j * 64 + i) % m.vocab for i in range(P.S)]
                      for j in range(P.K)], dtype=np.int32)
    return draft, grams


class GpuWorkload:
    def __init__(self, device, cache_len):
        from paper_2402_13720_b200 import binding, build
        build.build()
        self.m, _, self.P, _ = synth.config("C2")
        if cache_len + self.P.block_max + 1 > self.m.max_seq:
            raise SystemExit("cache length does not fit the configuration's max_seq")
        self.L = cache_len
        self.w = synth.model_weights(self.m, SEED, device=device)
        self.eng = binding.Engine(self.m, self.w, self.P, device=device)
        k, v = synth.kv_fill(self.m, SEED + 1, cache_len, device=device)
        self.eng.tm.k_cache.copy_(k)
        self.eng.tm.v_cache.copy_(v)
        self.draft, self.grams = block_inputs(self.m, self.P)
        self.eng.phrase_update(self.grams)
        self.eng.draft_tokens.copy_(torch.as_tensor(self.draft, device=device))
        self.draft_pinned = torch.as_tensor(self.draft).pin_memory()
        self.B = self.P.block_max
        self.bytes = algorithmic_bytes(self.m, self.B, self.L)

    def step(self, host_inputs=False):
        e = self.eng
        e.set_state(self.L, PENDING)
        if host_inputs:                               # end-to-end: the step's inputs start in pinned host memory
            e.draft_tokens.copy_(self.draft_pinned, non_blocking=True)
        return e.verify_step()                        # lookup + packing, forward, acceptance + compaction + harvest;
                                                      # returns host values: a device->host read per step

    def check(self):
        e = self.eng
        e.set_state(self.L, PENDING)
        e.assemble_candidates()
        assert e.block_get()[0].shape[0] == self.B, "the pool no longer yields K candidates"
        e.verify_forward()
        n, chosen, A, acc = e.accept_and_compact()
        assert 1 <= n <= self.P.gamma + self.P.beta
        return n


# -------------------------------------------------------------------------------- clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz, self._stop = [], set(), None, threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None
        self.t = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20,
                 "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(0.02)

    def __enter__(self):
        if self.nv:
            self.t.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self.nv:
            self.t.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}


# ------------------------------------------------------------------------------ CPU oracle

class OracleWorkload:
    """The same step on the CPU oracle, as it stands (numpy fp64)."""

    def __init__(self, cache_len):
        from oracle import ouroboros as ob, transformer as tf
        self.ob, self.tf = ob, tf
        self.m, _, self.P, _ = synth.config("C2")
        dev = "cuda:0" if torch.cuda.is_available() else "cpu"       # the generator is device independent
        w = synth.model_weights(self.m, SEED, device=dev)
        self.W = tf.Weights(self.m, w)
        k, v = synth.kv_fill(self.m, SEED + 1, cache_len, device=dev)
        self.cache = tf.KVCache(self.m, k.double().cpu().numpy(), v.double().cpu().numpy(), cache_len)
        self.L = cache_len
        self.draft, self.grams = block_inputs(self.m, self.P)
        self.pool = ob.PhrasePool(self.P.pool_sets, self.P.pool_ways, self.P.beta)
        for g in self.grams:
            self.pool.insert(g)
        self.bytes = algorithmic_bytes(self.m, self.P.block_max, cache_len)

    def step(self):
        ob, tf, P = self.ob, self.tf, self.P
        self.cache.length = self.L
        d = self.draft.tolist()
        cands = self.pool.lookup(d[-1], P.K)
        tokens, pos, group, vis = ob.build_block(self.L, PENDING, d, cands)
        o = tf.argmax_rows(tf.forward(self.W, self.cache, tokens, pos, vis))
        A, j, m, acc = ob.accept(tokens, o, P.gamma, P.S, len(cands))
        ob.compact(self.cache, self.L, P.gamma, P.S, A, j, m)
        seq = [0] * self.L + [PENDING] + acc
        self.pool.apply(ob.harvest_ops(tokens, o, P.gamma, P.S, len(cands), A, seq, len(acc), P))
        return acc


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


def time_oracle(cache_len, budget_s, max_steps=None):
    wl = OracleWorkload(cache_len)
    wl.step()
    t0 = time.perf_counter()
    n = 0
    while True:
        wl.step()
        n += 1
        el = time.perf_counter() - t0
        if el > budget_s or (max_steps and n >= max_steps):
            break
    return wl.bytes["total"] * n / el / 1e9, n, el


# ----------------------------------------------------------------------------------- main

def run_reference(args, rank):
    if rank != 0:
        return
    total = args.steps + args.warmup
    gbs, n, el = time_oracle(args.cache_len, 150.0 * args.steps / max(1, total), max_steps=args.steps)
    cores = blas_threads()
    sample = f"{n} of {args.steps} steps of the full workload executed ({el:.1f} s), rate taken over those"
    line = {"impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": el / n * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(args.cache_len),
            "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def workload_config(cache_len):
    return {"workload": "configs[1]: one 7B-shaped decoder layer + LM head, bf16, verify block of 37 rows "
                        "(1 + 4 draft + 4 phrases x 8)", "cache_len": cache_len, "block_rows": 37, "gamma": 4, "beta": 9,
            "K": 4, "vocab": 32000, "l2": "inputs (734 MB per step) larger than L2, each byte read once per step",
            "parallelism": "replicas"}


def run_generate(args, device):
    """End-to-end generation at batch 1: tokens/s of plain greedy decoding and of Ouroboros on the same GPU
    kernels.  Drafts: "natural" = the draft model's own greedy tokens (random-init pairs agree at chance level);
    "replay" = the target's recorded text with seeded substitutions and skips, standing in for a trained draft
    model at three agreement levels (the draft model's forwards still run and are timed)."""
    import dataclasses
    from paper_2402_13720_b200 import binding, build
    build.build()
    T, D, P, R = synth.config(args.generate)
    gen = args.gen_tokens or R["gen"]
    need = R["n"] + gen + P.block_max + 8
    T, D = dataclasses.replace(T, max_seq=max(T.max_seq, need)), dataclasses.replace(D, max_seq=max(D.max_seq, need))
    wt = synth.model_weights(T, SEED, device=device)
    wd = wt if args.generate == "C1" else synth.model_weights(D, SEED + 100, device=device)
    eng = binding.Engine(T, wt, P, D, wd, device=device)
    prompt = synth.prompt(SEED, T.vocab, R["n"], R["copy_frac"], *R["span"])
    eng.generate_vanilla(prompt, min(gen, 16))                                    # warm-up
    van, vs = eng.generate_vanilla(prompt, gen)
    res = {"vanilla": {"tokens_per_s": len(van) / (vs["ms_total"] * 1e-3), "ms_per_token": vs["ms_total"] / len(van)}}
    truth = np.concatenate([prompt, van, np.zeros(64, dtype=np.int32)])

    def run(name, drafter):
        eng.set_drafter(drafter)
        out, st = eng.generate(prompt, gen)
        eng.set_drafter(None)
        res[name] = {"tokens_per_s": len(out) / (st["ms_total"] * 1e-3), "tokens_per_target_call": len(out) / st["target_calls"],
                     "target_calls": st["target_calls"], "draft_calls": st["draft_calls"], "suffix_tokens": st["suffix_tokens"],
                     "ms_target_per_call": st["ms_target"] / st["target_calls"],
                     "ms_draft_per_step": st["ms_draft"] / st["target_calls"],
                     "identical_to_vanilla": bool(np.array_equal(out, van))}

    run("natural", None)
    for name, (ps, pk) in {"replay_low": (0.30, 0.05), "replay_mid": (0.12, 0.03), "replay_high": (0.04, 0.01)}.items():
        run(name, lambda seq, g, step, ps=ps, pk=pk: synth.corrupt_drafts(SEED + 7, truth, len(seq), g, T.vocab, ps, pk, step))

    # A random-init target does not repeat its prompt, so the pool (filled from the prompt and the accepted text)
    # rarely holds a phrase that starts with the draft's last token.  The paper's main phrase source, n-grams
    # produced during the draft model's forwards (Section 3.1), is not specified there; this stand-in feeds the pool
    # each step with K phrases that continue the draft: the recorded text after it, corrupted like the drafts.
    def with_phrases(seq, g, step):
        d = synth.corrupt_drafts(SEED + 7, truth, len(seq), g, T.vocab, 0.12, 0.03, step)
        grams = np.empty((P.K, P.beta), dtype=np.int32)
        for j in range(P.K):
            grams[j, 0] = d[-1]
            grams[j, 1:] = synth.corrupt_drafts(SEED + 11 + j, truth, len(seq) + g, P.S, T.vocab, 0.08 * (j + 1), 0.0, step)
        eng.phrase_update(grams[::-1])                      # the least corrupted phrase is inserted last = looked up first
        return d

    run("replay_mid_phrases", with_phrases)
    e = 2 if T.dtype == "bf16" else 4
    wbytes = T.n_layers * T.layer_weight_elems() * e + T.vocab * T.d_model * e
    peaks = {}
    # Phrase-level drafting on the draft model (Section 3.1): same weights and caches of their own, the draft model's
    # own drafts.  What changes is the number of draft forwards per target call (gamma / c of Eq. 6); with
    # random-init models c stays near 1 unless the draft model's text repeats.
    eng2 = binding.Engine(T, wt, dataclasses.replace(P, draft_phrases=True), D, wd, device=device)
    out, st = eng2.generate(prompt, gen)
    res["natural_phrase_drafting"] = {
        "tokens_per_s": len(out) / (st["ms_total"] * 1e-3), "target_calls": st["target_calls"], "draft_calls": st["draft_calls"],
        "draft_forwards_per_target_call": st["draft_calls"] / st["target_calls"],
        "ms_draft_per_step": st["ms_draft"] / st["target_calls"], "identical_to_vanilla": bool(np.array_equal(out, van))}
    eng2.close()
    # Phrase generation during the draft forward (Section 3.1): a lookahead window rides along every draft forward and
    # feeds the pool on the device; nothing is injected from the host.  With a random-init pair the draft model's
    # continuations rarely are the target's, so this run shows the cost of the window and whether candidates come up;
    # the acceptance of such phrases is shown where the draft model is the target itself (tests, C1).
    Pw = dataclasses.replace(P, window=max(P.S + 2, 12))
    eng3 = binding.Engine(T, wt, Pw, D, wd, device=device)
    out, st = eng3.generate(prompt, gen)
    res["natural_lookahead_window"] = {
        "window": Pw.window, "tokens_per_s": len(out) / (st["ms_total"] * 1e-3), "target_calls": st["target_calls"],
        "candidates": st["candidates"], "suffix_tokens": st["suffix_tokens"],
        "ms_draft_per_step": st["ms_draft"] / st["target_calls"], "identical_to_vanilla": bool(np.array_equal(out, van))}
    # History reuse (Section 3.4): the pool of earlier queries is kept for the next one.  Replayed drafts at the middle
    # agreement level, nothing injected from the host: the phrases come from the accepted text of the earlier run
    # (extension OURO_HARVEST_ACCEPTED) and from the verification's own corrections.  The same query again finds its
    # own continuation in the pool; another query finds little (synthetic texts share no phrases), which is the case
    # the paper's Table on context locality contrasts.
    mid = lambda truth_: (lambda seq, g, step: synth.corrupt_drafts(SEED + 7, truth_, len(seq), g, T.vocab, 0.12, 0.03, step))
    other = synth.prompt(SEED + 1, T.vocab, R["n"], R["copy_frac"], *R["span"])
    van_o, _ = eng.generate_vanilla(other, gen)
    truth_o = np.concatenate([other, van_o, np.zeros(64, dtype=np.int32)])
    eng.set_drafter(mid(truth))
    cold, stc = eng.generate(prompt, gen)
    warm, stw = eng.generate(prompt, gen, keep_pool=True)
    eng.set_drafter(mid(truth_o))
    o_cold, sto_c = eng.generate(other, gen)
    eng.set_drafter(mid(truth))
    eng.generate(prompt, gen)
    eng.set_drafter(mid(truth_o))
    o_warm, sto_w = eng.generate(other, gen, keep_pool=True)
    eng.set_drafter(None)
    tps = lambda o, st_: round(len(o) / (st_["ms_total"] * 1e-3), 1)
    res["history_reuse"] = {
        "drafts": "replay_mid",
        "same_query": {"cold_tokens_per_s": tps(cold, stc), "warm_tokens_per_s": tps(warm, stw),
                       "cold_target_calls": stc["target_calls"], "warm_target_calls": stw["target_calls"],
                       "cold_suffix_tokens": stc["suffix_tokens"], "warm_suffix_tokens": stw["suffix_tokens"],
                       "identical": bool(np.array_equal(cold, warm) and np.array_equal(cold, van))},
        "other_query": {"cold_tokens_per_s": tps(o_cold, sto_c), "warm_tokens_per_s": tps(o_warm, sto_w),
                        "cold_target_calls": sto_c["target_calls"], "warm_target_calls": sto_w["target_calls"],
                        "warm_suffix_tokens": sto_w["suffix_tokens"],
                        "identical": bool(np.array_equal(o_cold, o_warm) and np.array_equal(o_cold, van_o))}}
    eng3.close()

    # Algorithm 1 of the paper's Appendix B: coordinate search of gamma, W and beta on the wall-clock time of this
    # generation (replayed drafts at the middle agreement level, the replayed phrase source, K = 3).
    tuned = None
    if args.tune:
        from paper_2402_13720_b200 import tune

        def clock(g, w_, b, k):
            Pv = dataclasses.replace(P, gamma=g, window=w_, beta=b, K=k)
            e4 = binding.Engine(T, wt, Pv, D, wd, device=device)

            def drafter(seq, gg, step):
                d = synth.corrupt_drafts(SEED + 7, truth, len(seq), gg, T.vocab, 0.12, 0.03, step)
                grams = np.empty((Pv.K, Pv.beta), dtype=np.int32)
                for j in range(Pv.K):
                    grams[j, 0] = d[-1]
                    grams[j, 1:] = synth.corrupt_drafts(SEED + 11 + j, truth, len(seq) + gg, Pv.S, T.vocab, 0.08 * (j + 1), 0.0, step)
                e4.phrase_update(grams[::-1])
                return d

            e4.set_drafter(drafter)
            o4, st4 = e4.generate(prompt, gen)
            e4.set_drafter(None)
            e4.close()
            assert np.array_equal(o4, van)
            return st4["ms_total"]

        g0, w0, b0, k0, hist = tune.heuristic_search(clock, args.task)
        tuned = {"task_type": args.task, "gamma": g0, "window": w0, "beta": b0, "K": k0,
                 "tokens_per_s": round(gen / (min(h[4] for h in hist) * 1e-3), 1),
                 "evaluations": [{"gamma": h[0], "window": h[1], "beta": h[2], "ms": round(h[4], 2)} for h in hist]}

    # Sweeps over the method's knobs (the paper's K study, its gamma / beta grid and its component ablation, on
    # synthetic inputs): replayed drafts at the middle agreement level plus the seeded phrase source, one engine
    # per setting on the same weights.
    sweep = {}
    if args.sweep:
        def one(Pv, phrases=True):
            e3 = binding.Engine(T, wt, Pv, D, wd, device=device)

            def drafter(seq, g, step):
                d = synth.corrupt_drafts(SEED + 7, truth, len(seq), g, T.vocab, 0.12, 0.03, step)
                if phrases and Pv.K > 0 and Pv.S > 0:
                    grams = np.empty((Pv.K, Pv.beta), dtype=np.int32)
                    for j in range(Pv.K):
                        grams[j, 0] = d[-1]
                        grams[j, 1:] = synth.corrupt_drafts(SEED + 11 + j, truth, len(seq) + g, Pv.S, T.vocab, 0.08 * (j + 1), 0.0, step)
                    e3.phrase_update(grams[::-1])
                return d

            e3.set_drafter(drafter)
            out, st = e3.generate(prompt, gen)
            e3.set_drafter(None)
            e3.close()
            return {"tokens_per_s": round(len(out) / (st["ms_total"] * 1e-3), 1),
                    "tokens_per_target_call": round(len(out) / st["target_calls"], 2),
                    "ms_target_per_call": round(st["ms_target"] / st["target_calls"], 3),
                    "identical_to_vanilla": bool(np.array_equal(out, van))}

        rp = dataclasses.replace
        sweep["K"] = {k: one(rp(P, K=k)) for k in (0, 1, 2, 4, 8, 12)}
        sweep["gamma"] = {g: one(rp(P, gamma=g)) for g in (2, 4, 6, 8, 12)}
        sweep["beta"] = {b: one(rp(P, beta=b)) for b in (3, 5, 9, 13)}
        sweep["components"] = {
            "token-level drafts only (K = 0)": one(rp(P, K=0), phrases=False),
            "+ phrases from the pool as harvested (no phrase source)": one(P, phrases=False),
            "+ seeded phrase source": one(P),
            "paper-pure harvest flags + phrase source": one(P.paper_pure()),
        }

    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak = peaks.get("hbm_gbs", 6650.0)
    mid = res["replay_mid"]
    line = {"metric": "generated_tokens_per_s_batch1", "value": mid["tokens_per_s"], "unit": "tokens/s", "n_gpus": 1,
            "higher_is_better": True, "dtype": T.dtype, "data": "synthetic",
            "config": {"workload": f"{args.generate}: prompt {R['n']}, generate {gen}, gamma {P.gamma}, beta {P.beta}, K {P.K}",
                       "drafts": "replay_mid (seeded corruption of the target's own text: p_sub 0.12, p_skip 0.03)"},
            "vs_vanilla": mid["tokens_per_s"] / res["vanilla"]["tokens_per_s"],
            "vanilla_ceiling_tokens_per_s": peak * 1e9 / wbytes,
            "verify_forward_gbs": wbytes / (mid["ms_target_per_call"] * 1e-3) / 1e9,
            "verify_forward_frac_of_peak": wbytes / (mid["ms_target_per_call"] * 1e-3) / 1e9 / peak,
            "with_phrases_vs_vanilla": res["replay_mid_phrases"]["tokens_per_s"] / res["vanilla"]["tokens_per_s"],
            "results": res}
    if sweep:
        line["sweep"] = sweep
    if tuned:
        line["algorithm1"] = tuned
    print(json.dumps(line))
    eng.close()


def generation_summary(device, tokens):
    """The metric's other half: generated tokens/s at batch 1 on the 7B-shaped target with the 1.1B-shaped draft model
    (configuration C3), plain greedy decoding against Ouroboros with replayed drafts (middle agreement level), the same
    with the pool of the run before (history reuse), and with the replayed phrase source.  A short run: `tokens` generated tokens per mode."""
    import dataclasses
    from paper_2402_13720_b200 import binding
    T, D, P, R = synth.config("C3")
    wt = synth.model_weights(T, SEED, device=device)
    wd = synth.model_weights(D, SEED + 100, device=device)
    eng = binding.Engine(T, wt, P, D, wd, device=device)
    prompt = synth.prompt(SEED, T.vocab, R["n"], R["copy_frac"], *R["span"])
    eng.generate_vanilla(prompt, 8)
    van, vs = eng.generate_vanilla(prompt, tokens)
    truth = np.concatenate([prompt, van, np.zeros(64, dtype=np.int32)])
    out = {"config": f"configs[2]: 7B-shaped target, 1.1B-shaped draft, bf16, prompt {R['n']}, {tokens} tokens, gamma {P.gamma}, "
                     f"beta {P.beta}, K {P.K}",
           "vanilla": {"tokens_per_s": round(len(van) / (vs["ms_total"] * 1e-3), 1)}}

    def run(name, drafter, keep_pool=False):
        eng.set_drafter(drafter)
        o, st = eng.generate(prompt, tokens, keep_pool=keep_pool)
        eng.set_drafter(None)
        out[name] = {"tokens_per_s": round(len(o) / (st["ms_total"] * 1e-3), 1),
                     "vs_vanilla": round(len(o) / (st["ms_total"] * 1e-3) / out["vanilla"]["tokens_per_s"], 3),
                     "tokens_per_target_call": round(len(o) / st["target_calls"], 2), "suffix_tokens": st["suffix_tokens"],
                     "ms_target_per_call": round(st["ms_target"] / st["target_calls"], 3),
                     "ms_draft_per_step": round(st["ms_draft"] / st["target_calls"], 3),
                     "identical_to_vanilla": bool(np.array_equal(o, van))}

    def drafts(seq, g, step):
        return synth.corrupt_drafts(SEED + 7, truth, len(seq), g, T.vocab, 0.12, 0.03, step)

    def drafts_and_phrases(seq, g, step):
        d = drafts(seq, g, step)
        grams = np.empty((P.K, P.beta), dtype=np.int32)
        for j in range(P.K):
            grams[j, 0] = d[-1]
            grams[j, 1:] = synth.corrupt_drafts(SEED + 11 + j, truth, len(seq) + g, P.S, T.vocab, 0.08 * (j + 1), 0.0, step)
        eng.phrase_update(grams[::-1])
        return d

    run("replayed_drafts", drafts)
    # Section 3.4, history reuse: the same query once more with the pool the run above left behind (nothing injected)
    run("replayed_drafts_warm_pool", drafts, keep_pool=True)
    run("replayed_drafts_and_phrases", drafts_and_phrases)
    eng.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cache-len", type=int, default=4096)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-generation", action="store_true", help="skip the short whole-model generation summary")
    ap.add_argument("--generation-tokens", type=int, default=96)
    ap.add_argument("--generate", default=None, choices=["C1", "C3", "C4", "C5"],
                    help="instead of the verify-step benchmark: whole generation on that configuration "
                         "(vanilla greedy vs Ouroboros, natural and replayed drafts), one JSON line")
    ap.add_argument("--sweep", action="store_true", help="with --generate: K, gamma, beta and component sweeps as well")
    ap.add_argument("--gen-tokens", type=int, default=0, help="override the configuration's generation length")
    ap.add_argument("--tune", action="store_true", help="with --generate: the paper's Algorithm 1 (coordinate search of "
                    "gamma, W, beta on wall-clock time)")
    ap.add_argument("--task", default="LH", choices=["HH", "LH"], help="recipe range of gamma for --tune")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        return run_reference(args, rank)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    from paper_2402_13720_b200 import binding, dist_util
    torch.cuda.set_device(local)
    device = f"cuda:{local}"
    if args.generate:
        return run_generate(args, device)
    group = dist_util.init(world, rank, "nccl") if world > 1 else None
    wl = GpuWorkload(device, args.cache_len)
    lib = binding.lib()
    for _ in range(max(3, args.warmup)):
        wl.check()
    stream = torch.cuda.current_stream()

    def timed(host_inputs):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        dist_util.barrier(group)
        torch.cuda.synchronize()
        launches0 = lib.ouro_kernel_launches()
        with ClockSampler(local) as cs:
            ev0.record(stream)
            for _ in range(args.steps):
                wl.step(host_inputs)
            ev1.record(stream)
            torch.cuda.synchronize()
        dist_util.barrier(group)
        ms = dist_util.max_over_ranks(ev0.elapsed_time(ev1), group)
        return ms, lib.ouro_kernel_launches() - launches0, cs.summary()

    ms, launches, clocks = timed(False)
    ms_e2e, _, _ = timed(True)
    total_bytes = dist_util.sum_over_ranks(wl.bytes["total"] * args.steps, group)   # every replica's units
    value = total_bytes / (ms * 1e-3) / 1e9
    e2e = total_bytes / (ms_e2e * 1e-3) / 1e9

    # per-kernel-class device time of the forward, events on the library's own stream.  "gemm" brackets every launch
    # of the weight-streaming kernel as the forward really runs it (two launches per step: q,k,v with the embedding
    # gather; output projection + gate/up + down + LM head as one chain).  The per-GEMM classes are diagnostics: while
    # one of them is timed, each GEMM is launched alone.
    prof = {}
    psteps = min(args.steps, 200)
    for cls in PROF_CLASSES + ("gemm", "forward"):
        wl.eng.profile_enable(cls)
        for _ in range(psteps):
            wl.step()
        t, n = wl.eng.profile_read()
        prof[cls] = (t / max(1, n), n // psteps)
    wl.eng.profile_enable("off")
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    peak, peak_kind = (peaks["hbm_gbs"], "measured") if "hbm_gbs" in peaks else (6650.0, "fallback")
    # The dominant kernel is the weight-streaming GEMM: its launches of one step stream every weight matrix once.
    gemm = ("qkv", "wo", "gateup", "down", "head")
    gemm_launches = prof["gemm"][1]
    gemm_ms = prof["gemm"][0] * gemm_launches
    gemm_bytes = sum(wl.bytes["per_class"][c] for c in gemm) * wl.m.n_layers - (wl.m.n_layers - 1) * wl.bytes["per_class"]["head"]
    achieved = gemm_bytes / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0
    fwd_ms = prof["forward"][0]
    # DRAM bytes per launch (read + write) from one ncu capture of this workload, kept in the tracked profile
    # summary; null once the kernel's device code has changed since the capture.
    traffic = profiled_traffic() if args.cache_len == 4096 else None
    roofline = {"bound": "hbm", "kernel": "gemm_tc_kernel", "launches_per_step": gemm_launches,
                "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic,
                "bytes_per_launch": gemm_bytes / max(1, gemm_launches), "us_per_launch": gemm_ms * 1e3 / max(1, gemm_launches),
                "kernel_us": {"gemm": round(prof["gemm"][0] * 1e3, 2), "attention": round(prof["attention"][0] * 1e3, 2)},
                "gemm_us_when_launched_alone": {c: round(prof[c][0] * 1e3, 2) for c in gemm},
                "forward_us": round(fwd_ms * 1e3, 2),
                "forward_gbs": wl.bytes["total"] / (fwd_ms * 1e-3) / 1e9 if fwd_ms > 0 else 0.0,
                "forward_frac": wl.bytes["total"] / (fwd_ms * 1e-3) / 1e9 / peak if fwd_ms > 0 else 0.0}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup),
            "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic", "config": workload_config(args.cache_len), "clocks": clocks,
            "e2e": {"value": e2e, "unit": UNIT, "h2d_bytes_per_step": int(wl.draft.nbytes),
                    "d2h_bytes_per_step": 220},   # acceptance record (216 B) + its sequence number
            "gpu_launches": int(launches), "roofline": roofline, "bytes_per_step": wl.bytes["total"]}
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        gbs, n, el = time_oracle(args.cache_len, 10.0)
        line["cpu_baseline"] = {"value": gbs, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                                "sample": f"{n} full steps of the same workload in {el:.1f} s"}
    if rank == 0 and world == 1 and not args.no_generation:
        wl.eng.close()
        del wl
        torch.cuda.empty_cache()
        line["generation"] = generation_summary(device, args.generation_tokens)
    if rank == 0:
        print(json.dumps(line))
    dist_util.finish(group)


if __name__ == "__main__":
    main()
