"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs.

Floating point: fp32 logits within 1e-3 max-abs; bf16 logits within 3e-2 of the row's largest |logit|.
Integers (block layout, acceptance, compaction indices, pool contents, tokens) are bit exact.
"""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import ouroboros as ob
from oracle import transformer as tf
from paper_2402_13720_b200 import binding, build, synth

pytestmark = pytest.mark.gpu

FP32_TOL = 1e-3
BF16_REL = 3e-2

TINY = synth.ModelDesc(2, 64, 4, 2, 32, 96, 100, 192, "f32")
MIDB = synth.ModelDesc(3, 256, 8, 2, 64, 512, 1000, 320, "bf16")     # GQA 4:1, head_dim 64, bf16
C1T, C1D, C1P, C1R = synth.config("C1")


@pytest.fixture(scope="module", autouse=True)
def _built():
    build.build()


def make(desc, params, seed=0, draft=None):
    """Engine on cuda:0 and the oracle's weights; the generator gives identical values on both devices."""
    w = synth.model_weights(desc, seed, device="cuda:0")
    eng = binding.Engine(desc, w, params, draft, w if draft is not None else None)
    return eng, tf.Weights(desc, synth.model_weights(desc, seed))


def test_generated_inputs_are_device_independent():
    a = synth.model_weights(MIDB, 7, device="cuda:0")
    b = synth.model_weights(MIDB, 7)
    assert torch.equal(a["lm_head"].cpu(), b["lm_head"]) and torch.equal(a["layers"][2]["w_down"].cpu(), b["layers"][2]["w_down"])
    assert torch.equal(a["layers"][0]["attn_norm"].cpu(), b["layers"][0]["attn_norm"])


def oracle_pool(P):
    return ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)


def pool_rows(pool):
    ex = pool.export()
    return [list(p) for _, p in ex], [s for s, _ in ex]


def gpu_pool_rows(eng):
    ng, st = eng.pool_export()
    return ng.tolist(), st.tolist()


# ------------------------------------------------------------------------------------ pool

@pytest.mark.parametrize("sets,ways,beta", [(4, 3, 3), (1, 2, 2), (8, 40, 5)])
def test_pool_matches_oracle(sets, ways, beta):
    P = synth.DecodeParams(2, beta, 3, sets, ways)
    eng, _ = make(TINY, P)
    ref = oracle_pool(P)
    rng = np.random.default_rng(sets * 100 + ways)
    for rnd in range(12):
        grams = rng.integers(0, 7, (int(rng.integers(1, 40)), beta))
        eng.phrase_update(grams)
        for g in grams:
            ref.insert(g)
        assert gpu_pool_rows(eng) == pool_rows(ref)
        for key in range(8):
            got = eng.phrase_lookup(key).tolist()
            assert got == ref.lookup(key, P.K)
            assert all(len(s) == beta - 1 for s in got)
    # export -> reset -> import reproduces the same retrieval order
    ng, _ = eng.pool_export()
    eng.reset(keep_pool=False)
    assert eng.pool_export()[0].shape[0] == 0 and eng.phrase_lookup(3).shape[0] == 0
    eng.pool_import(ng)
    for key in range(8):
        assert eng.phrase_lookup(key).tolist() == ref.lookup(key, P.K)
    eng.close()


# ------------------------------------------------------------------------- candidate packing

@pytest.mark.parametrize("gamma,beta,K,n_fill", [(4, 4, 4, 60), (3, 9, 4, 80), (2, 3, 0, 10), (5, 6, 3, 0), (1, 2, 16, 50)])
def test_assemble_matches_oracle(gamma, beta, K, n_fill):
    P = synth.DecodeParams(gamma, beta, K, 4, 8, seed_prompt=False)
    eng, _ = make(TINY, P)
    ref = oracle_pool(P)
    rng = np.random.default_rng(gamma * 10 + beta)
    if n_fill:
        grams = rng.integers(0, 5, (n_fill, beta))
        eng.phrase_update(grams)
        for g in grams:
            ref.insert(g)
    prompt = rng.integers(0, TINY.vocab, 21).astype(np.int32)
    eng.prefill(prompt)
    L = len(prompt) - 1
    for trial in range(4):
        d = rng.integers(0, 5, gamma).tolist()
        eng.assemble_candidates(draft=d)
        tok, pos, grp, mask = eng.block_get()
        cands = ref.lookup(d[-1], K)
        t2, p2, g2, vis = ob.build_block(L, prompt[-1], d, cands)
        assert tok.tolist() == t2 and pos.tolist() == p2 and grp.tolist() == g2
        B = len(t2)
        bits = np.array([[(int(mask[r, c // 64]) >> (c % 64)) & 1 for c in range(B)] for r in range(B)], dtype=bool)
        assert np.array_equal(bits, vis[:, L:])
        assert all(c[0] is not None for c in cands) and B == 1 + gamma + len(cands) * (beta - 1)
        # the same block through an explicit lookup
        got = eng.phrase_lookup(d[-1])
        eng.assemble_candidates(draft=d, lookup_here=False)
        assert eng.block_get()[0].tolist() == t2 and got.tolist() == cands
    eng.close()


# ------------------------------------------------------------------------------ forward logits

def _verify_case(eng, W, desc, P, seed, L_prompt, tol_fn, full_block=False):
    rng = np.random.default_rng(seed)
    prompt = synth.prompt(seed, desc.vocab, L_prompt, 0.4, 4, 8)
    eng.reset()
    eng.prefill(prompt)
    ref_pool = oracle_pool(P)
    ref_pool.apply(ob.prompt_ops(prompt, P.beta, P))
    d = rng.integers(0, desc.vocab, P.gamma).tolist()
    d[-1] = int(prompt[5])                     # a key that the seeded pool knows
    if full_block:                             # K phrases with that key, so that the block has all its rows
        grams = rng.integers(0, desc.vocab, (P.K, P.beta)).astype(np.int32)
        grams[:, 0] = d[-1]
        eng.phrase_update(grams)
        for g in grams:
            ref_pool.insert(g)
    eng.assemble_candidates(draft=d)
    tok, pos, grp, mask = eng.block_get()
    cands = ref_pool.lookup(d[-1], P.K)
    t2, p2, g2, vis = ob.build_block(len(prompt) - 1, prompt[-1], d, cands)
    assert tok.tolist() == t2 and len(cands) >= 1 and (not full_block or len(t2) == P.block_max)
    am, logits = eng.verify_forward(want_logits=True)
    cache = tf.KVCache(desc)
    ob.prefill(W, cache, list(prompt[:-1]))
    L = cache.length
    want = tf.forward(W, cache, t2, p2, vis)
    got = logits[: len(t2)].cpu().numpy().astype(np.float64)
    tol_fn(got, want)
    # greedy choice agrees wherever the oracle's top-2 margin exceeds the numeric error
    err = np.abs(got - want).max(axis=1)
    srt = np.sort(want, axis=1)
    safe = (srt[:, -1] - srt[:, -2]) > 2 * err + 1e-12
    assert safe.sum() >= 1
    assert np.array_equal(am[: len(t2)].cpu().numpy()[safe], tf.argmax_rows(want)[safe])
    # K/V appended by the forward equal the oracle's (cache slots L .. L+B-1 of every layer)
    k_gpu = eng.tm.k_cache[:, : L + len(t2)].float().cpu().numpy()
    v_gpu = eng.tm.v_cache[:, : L + len(t2)].float().cpu().numpy()
    kv_tol = 1e-4 if desc.dtype == "f32" else 2e-2 * max(np.abs(cache.k).max(), np.abs(cache.v).max())
    assert np.abs(k_gpu - cache.k[:, : L + len(t2)]).max() < kv_tol
    assert np.abs(v_gpu - cache.v[:, : L + len(t2)]).max() < kv_tol


def _fp32_tol(got, want):
    assert np.abs(got - want).max() < FP32_TOL


def _bf16_tol(got, want):
    rel = np.abs(got - want).max(axis=1) / np.abs(want).max(axis=1)
    assert rel.max() < BF16_REL, rel.max()


@pytest.mark.parametrize("seed,L_prompt", [(0, 32), (1, 33), (2, 130), (3, 9)])
def test_verify_logits_fp32_c1(seed, L_prompt):
    eng, W = make(C1T, C1P, seed)
    _verify_case(eng, W, C1T, C1P, seed, L_prompt, _fp32_tol)
    eng.close()


@pytest.mark.parametrize("seed,L_prompt", [(0, 40), (1, 257)])
def test_verify_logits_bf16(seed, L_prompt):
    P = synth.DecodeParams(4, 9, 4, 16, 8)
    eng, W = make(MIDB, P, seed)
    _verify_case(eng, W, MIDB, P, seed, L_prompt, _bf16_tol)
    eng.close()


def test_packed_block_equals_separate_causal_forwards_on_gpu():
    """Eq. 8 on the GPU itself, bit for bit: a suffix row's logits equal those of the same token decoded
    as plain causal text (which is what makes the method lossless on this library)."""
    P = synth.DecodeParams(3, 4, 2, 4, 8, seed_prompt=False)
    eng, _ = make(MIDB, P, 5)
    rng = np.random.default_rng(5)
    prompt = rng.integers(0, MIDB.vocab, 70).astype(np.int32)
    d = rng.integers(0, MIDB.vocab, 3).tolist()
    cands = rng.integers(0, MIDB.vocab, (2, 3))
    eng.phrase_update(np.concatenate([np.full((2, 1), d[-1]), cands], axis=1))
    eng.prefill(prompt)
    eng.assemble_candidates(draft=d)
    tok = eng.block_get()[0]
    assert len(tok) == 10
    _, logits = eng.verify_forward(want_logits=True)
    packed = logits[:10].clone()
    order = [tok[4:7].tolist(), tok[7:10].tolist()]
    for j, suffix in enumerate(order):
        eng.reset()
        eng.prefill(prompt)
        lin = [int(prompt[-1])] + d + suffix
        rows = []
        for t in lin:                                  # one token per forward, like plain decoding
            eng.assemble_causal(binding.OURO_TARGET, [t])
            _, lg = eng.verify_forward(want_logits=True)
            rows.append(lg[0].clone())
            eng.advance(binding.OURO_TARGET, 1)
        rows = torch.stack(rows)
        assert torch.equal(rows[:4], packed[:4])
        assert torch.equal(rows[4:], packed[4 + 3 * j: 7 + 3 * j])
    eng.close()


# ------------------------------------------------------------- acceptance, compaction, harvest

def _hand_trace(name):
    from test_oracle_ouroboros import load_trace
    return load_trace(name)


@pytest.mark.parametrize("name", ["trace_partial_accept.txt", "trace_full_accept.txt", "trace_tie.txt"])
def test_hand_traces_on_gpu(name):
    t = _hand_trace(name)
    gamma, beta = t["gamma"], t["beta"]
    P = synth.DecodeParams(gamma, beta, max(1, len(t["candidates"])), 8, 4, harvest_accepted=False, seed_prompt=False)
    eng, _ = make(TINY, P)
    for c in t["candidates"]:
        eng.phrase_update([[t["draft"][-1]] + c])
    prompt = np.array([1, 2, 3, 4, 5, 6, 7, t["pending"]], dtype=np.int32)
    eng.prefill(prompt)
    # candidates come back newest first; the traces list them in block order
    eng.count.fill_(len(t["candidates"]))
    if t["candidates"]:
        eng.suffix[: len(t["candidates"]) * (beta - 1)] = torch.tensor(np.array(t["candidates"]).ravel(), dtype=torch.int32, device="cuda")
    eng.assemble_candidates(draft=t["draft"], lookup_here=False)
    eng.verify_forward()
    o = torch.tensor(t["outputs"], dtype=torch.int32, device="cuda")
    n, chosen, A, acc = eng.accept_and_compact(o)
    assert (A, chosen, acc.tolist()) == (t["A"], t["chosen"], t["accepted"]) and n == len(t["accepted"])
    assert eng.get_state()[0] == 7 + t["new_length_minus_L"] and eng.get_state()[2] == t["accepted"][-1]
    if "pool_after" in t:
        assert gpu_pool_rows(eng)[0] == t["pool_after"]
    if "ops_matched_only" in t:
        assert gpu_pool_rows(eng)[0] == [op[1] for op in t["ops_matched_only"]]
    eng.close()


@pytest.mark.parametrize("gamma,beta,K,flags", [
    (4, 4, 4, {}), (3, 3, 2, {}), (2, 9, 4, {}), (5, 2, 3, {}), (4, 4, 0, {}),
    (4, 4, 4, dict(harvest_accepted=False, seed_prompt=False)),
    (6, 3, 3, dict(harvest_candidates=False)), (4, 5, 4, dict(harvest_matched=False, harvest_accepted=False))])
def test_accept_compact_harvest_fuzz(gamma, beta, K, flags):
    """Random verification outcomes injected as the argmax vector: every integer result, the moved KV rows
    and the pool contents must equal the oracle's, step after step."""
    P = synth.DecodeParams(gamma, beta, K, 4, 6, **flags)
    S = beta - 1
    eng, _ = make(TINY, P)
    rng = np.random.default_rng(gamma * 100 + beta * 10 + K)
    V = 4                                                     # tiny alphabet: matches happen all the time
    prompt = rng.integers(0, V, 12).astype(np.int32)
    eng.prefill(prompt)
    pool = oracle_pool(P)
    pool.apply(ob.prompt_ops(prompt, beta, P))
    seq = prompt.tolist()
    moved = full = 0
    for step in range(40):
        L = len(seq) - 1
        assert eng.get_state()[0] == L and eng.get_state()[2] == seq[-1]
        d = rng.integers(0, V, gamma).tolist()
        cands = pool.lookup(d[-1], K)
        eng.assemble_candidates(draft=d)
        tokens, pos, group, vis = ob.build_block(L, seq[-1], d, cands)
        assert eng.block_get()[0].tolist() == tokens
        B = len(tokens)
        eng.verify_forward()
        torch.cuda.synchronize()
        k_before = eng.tm.k_cache.clone(); v_before = eng.tm.v_cache.clone()
        # outputs that agree with the row's successor most of the time
        o = rng.integers(0, V, B)
        for b in range(B):
            if rng.random() < 0.8:
                if b < gamma:
                    o[b] = tokens[b + 1]
                elif b == gamma and cands:
                    o[b] = cands[int(rng.integers(0, len(cands)))][0]
                elif b > gamma and (b - gamma) % S != 0:          # not the last row of its suffix
                    o[b] = tokens[b + 1]
        o_dev = torch.tensor(o, dtype=torch.int32, device="cuda")
        n, chosen, A, acc = eng.accept_and_compact(o_dev)
        A2, j2, m2, acc2 = ob.accept(tokens, o.tolist(), gamma, S, len(cands))
        assert (n, chosen, A, acc.tolist()) == (len(acc2), j2, A2, acc2)
        # compaction: expected cache = before + the oracle's moves
        cache = tf.KVCache(dataclasses.replace(TINY, n_layers=1, max_seq=TINY.max_seq))
        cache.length = L
        moves = ob.compact(cache, L, gamma, S, A2, j2, m2)
        k_exp, v_exp = k_before.clone(), v_before.clone()
        for s, dst in moves:
            k_exp[:, dst] = k_before[:, s]; v_exp[:, dst] = v_before[:, s]
        Ln = cache.length
        assert torch.equal(eng.tm.k_cache[:, :Ln], k_exp[:, :Ln]) and torch.equal(eng.tm.v_cache[:, :Ln], v_exp[:, :Ln])
        moved += len(moves); full += A2 == gamma
        seq += acc2
        pool.apply(ob.harvest_ops(tokens, o.tolist(), gamma, S, len(cands), A2, seq, len(acc2), P))
        assert gpu_pool_rows(eng) == pool_rows(pool)
        if len(seq) + P.block_max + 1 >= TINY.max_seq:
            break
    assert full > 3 and (moved > 0 or K < 2 or S == 0)
    eng.close()


# -------------------------------------------------------------------------- end to end (C1)

@pytest.fixture(scope="module")
def c1():
    w = synth.model_weights(C1T, 0, device="cuda:0")
    eng = binding.Engine(C1T, w, C1P, C1D, w)
    W = tf.Weights(C1T, synth.model_weights(C1T, 0))
    yield eng, W, tf.Weights(C1D, synth.model_weights(C1T, 0))
    eng.close()


C1_SEEDS = [0, 1, 2, 4]
_c1_seen = {}


@pytest.mark.parametrize("seed", C1_SEEDS)
def test_generate_c1_matches_oracle_and_vanilla(c1, seed):
    eng, W, Wd = c1
    prompt = synth.prompt(seed, C1T.vocab, C1R["n"], C1R["copy_frac"], *C1R["span"])
    gen = C1R["gen"]
    out, stats = eng.generate(prompt, gen)
    pool_gpu = gpu_pool_rows(eng)
    van, vstats = eng.generate_vanilla(prompt, gen)
    assert np.array_equal(out, van)                                   # lossless on the GPU, bit for bit
    assert vstats["target_calls"] == gen and stats["target_calls"] <= gen
    trace = []
    ref, rstats = ob.generate(W, ob.ModelDrafter(Wd), prompt, gen, C1P, trace=trace)
    assert out.tolist() == ref                                        # and equal to the oracle's text
    assert stats["target_calls"] == rstats["target_calls"]
    assert stats["full_accepts"] == sum(a == C1P.gamma for a in rstats["A"])
    assert stats["suffix_tokens"] == sum(rstats["m"])
    assert stats["candidates"] == sum(rstats["n_cand"])
    assert pool_gpu[0] == [list(p) for _, p in trace[-1]["pool"]]    # same pool, same order
    assert pool_gpu[1] == [s for s, _ in trace[-1]["pool"]]
    _c1_seen[seed] = (sum(rstats["A"]), stats["suffix_tokens"], stats["target_calls"])
    if len(_c1_seen) == len(C1_SEEDS):
        # The early-exit draft (one of the target's two layers) agrees with the target only now and then: seed 0 runs
        # with block efficiency 1 (no draft token is ever accepted).  Over the seeds draft tokens must have been
        # accepted, or this comparison would not exercise acceptance at all.  Phrase suffixes are never accepted
        # with these natural drafts; the replayed-draft test below asserts suffix_tokens > 0.
        assert sum(v[0] for v in _c1_seen.values()) > 20, _c1_seen
        assert any(v[2] < gen for v in _c1_seen.values()), _c1_seen


def test_teacher_forced_steps_c1(c1):
    """Step the GPU through its own API; at every step the oracle evaluates the same block on the same
    history: logits within tolerance, integer results and pool bit exact."""
    eng, W, Wd = c1
    P = C1P
    prompt = synth.prompt(4, C1T.vocab, 32, 0.5, 8, 8)
    eng.reset(); eng.prefill(prompt)
    cache = tf.KVCache(C1T); ob.prefill(W, cache, list(prompt[:-1]))
    pool = oracle_pool(P); pool.apply(ob.prompt_ops(prompt, P.beta, P))
    seq = prompt.tolist()
    for step in range(12):
        L = cache.length
        d = eng.draft().cpu().numpy()[: P.gamma].tolist()
        eng.assemble_candidates()
        tok = eng.block_get()[0].tolist()
        cands = pool.lookup(d[-1], P.K)
        tokens, pos, group, vis = ob.build_block(L, seq[-1], d, cands)
        assert tok == tokens
        am, logits = eng.verify_forward(want_logits=True)
        want = tf.forward(W, cache, tokens, pos, vis)
        assert np.abs(logits[: len(tokens)].cpu().numpy() - want).max() < FP32_TOL
        o = am[: len(tokens)].cpu().numpy().tolist()
        n, chosen, A, acc = eng.accept_and_compact()
        A2, j2, m2, acc2 = ob.accept(tokens, o, P.gamma, P.S, len(cands))
        assert (n, chosen, A, acc.tolist()) == (len(acc2), j2, A2, acc2)
        ob.compact(cache, L, P.gamma, P.S, A2, j2, m2)
        seq += acc2
        pool.apply(ob.harvest_ops(tokens, o, P.gamma, P.S, len(cands), A2, seq, len(acc2), P))
        assert gpu_pool_rows(eng) == pool_rows(pool)
        Ln = cache.length
        assert np.abs(eng.tm.k_cache[:, :Ln].cpu().numpy() - cache.k[:, :Ln]).max() < 1e-4
        assert np.abs(eng.tm.v_cache[:, :Ln].cpu().numpy() - cache.v[:, :Ln]).max() < 1e-4


def test_external_drafter_replay_is_lossless(c1):
    eng, W, _ = c1
    prompt = synth.prompt(9, C1T.vocab, 32, 0.5, 8, 8)
    van, _ = eng.generate_vanilla(prompt, 64)
    truth = np.concatenate([prompt, van, np.zeros(16, dtype=np.int32)])
    eng.set_drafter(lambda seq, g, step: synth.corrupt_drafts(3, truth, len(seq), g, C1T.vocab, 0.05, 0.05, step))
    try:
        out, stats = eng.generate(prompt, 64)
        pool_gpu = gpu_pool_rows(eng)
    finally:
        eng.set_drafter(None)
    assert np.array_equal(out, van)
    drafter = ob.FixedDrafter(lambda seq, g, step: synth.corrupt_drafts(3, truth, len(seq), g, C1T.vocab, 0.05, 0.05, step))
    trace = []
    ref, rstats = ob.generate(W, drafter, prompt, 64, C1P, trace=trace)
    assert out.tolist() == ref and stats["target_calls"] == rstats["target_calls"]
    assert stats["suffix_tokens"] == sum(rstats["m"]) > 0
    assert pool_gpu[0] == [list(p) for _, p in trace[-1]["pool"]]


def test_history_reuse_and_eos(c1):
    eng, W, Wd = c1
    p1 = synth.prompt(10, C1T.vocab, 24, 0.5, 8, 8)
    p2 = synth.prompt(11, C1T.vocab, 24, 0.5, 8, 8)
    eng.generate(p1, 24)
    n1 = eng.pool_export()[0].shape[0]
    out2, _ = eng.generate(p2, 24, keep_pool=True)                    # Section 3.4: the pool survives the query
    assert eng.pool_export()[0].shape[0] > 0 and n1 > 0
    assert np.array_equal(out2, eng.generate_vanilla(p2, 24)[0])
    pool = oracle_pool(C1P)
    for p in (p1, p2):
        ref, _ = ob.generate(W, ob.ModelDrafter(Wd), p, 24, C1P, pool=pool)
    eng.generate(p1, 24); eng.generate(p2, 24, keep_pool=True)
    assert gpu_pool_rows(eng)[0] == pool_rows(pool)[0]
    # stop token
    van, _ = eng.generate_vanilla(p1, 24)
    eos = int(van[7])
    Pe = dataclasses.replace(C1P, eos_token=eos)
    w = synth.model_weights(C1T, 0, device="cuda:0")
    e2 = binding.Engine(C1T, w, Pe, C1D, w)
    cut = van[: van.tolist().index(eos) + 1]
    assert np.array_equal(e2.generate(p1, 24)[0], cut) and np.array_equal(e2.generate_vanilla(p1, 24)[0], cut)
    e2.close()


# ------------------------------------------------------------------ lossless in bf16, edge cases

def test_bf16_ouroboros_is_bit_identical_to_vanilla():
    P = synth.DecodeParams(4, 9, 4, 32, 8)
    eng, _ = make(MIDB, P, 3)
    prompt = synth.prompt(3, MIDB.vocab, 96, 0.3, 8, 32)
    van, _ = eng.generate_vanilla(prompt, 160)
    truth = np.concatenate([prompt, van, np.zeros(32, dtype=np.int32)])
    for p_sub in (0.0, 0.15):
        eng.set_drafter(lambda seq, g, step: synth.corrupt_drafts(1, truth, len(seq), g, MIDB.vocab, p_sub, 0.05, step))
        out, stats = eng.generate(prompt, 160)
        assert np.array_equal(out, van)
        assert stats["target_calls"] < 160 and stats["suffix_tokens"] > 0
    eng.set_drafter(None)
    eng.close()


def test_edge_cases():
    P = synth.DecodeParams(4, 4, 4, 8, 4)
    eng, W = make(TINY, P)
    # a one-token prompt: nothing to prefill, the pool stays empty at first
    out, _ = eng.generate_vanilla(np.array([5], dtype=np.int32), 6)
    assert out.tolist() == ob.vanilla_greedy(W, [5], 6)
    # capacity: the cache cannot take prompt + block
    with pytest.raises(binding.OuroError) as e:
        eng.reset(); eng.prefill(np.zeros(TINY.max_seq - 3, dtype=np.int32))
    assert e.value.status == binding.OURO_ECAPACITY
    # call order: verify without a block, accept without a verification
    eng.reset(); eng.prefill(np.array([1, 2, 3], dtype=np.int32))
    with pytest.raises(binding.OuroError) as e:
        eng.verify_forward()
    assert e.value.status == binding.OURO_ESTATE
    with pytest.raises(binding.OuroError) as e:
        eng.accept_and_compact()
    assert e.value.status == binding.OURO_ESTATE
    # no draft model and no drafter
    with pytest.raises(binding.OuroError):
        eng.draft()
    # token out of range
    with pytest.raises(binding.OuroError) as e:
        eng.reset(); eng.prefill(np.array([1, TINY.vocab], dtype=np.int32))
    assert e.value.status == binding.OURO_EINVAL
    # widest block the library takes: 1 + 7 + 8*15 = 128 rows
    Pw = synth.DecodeParams(7, 16, 8, 2, 16, seed_prompt=False)
    e2, W2 = make(TINY, Pw, 1)
    grams = np.random.default_rng(0).integers(0, TINY.vocab, (8, 16)); grams[:, 0] = 9
    e2.phrase_update(grams)
    prompt = synth.prompt(0, TINY.vocab, 20, 0.0, 4, 4)
    e2.prefill(prompt)
    d = [1, 2, 3, 4, 5, 6, 9]
    e2.assemble_candidates(draft=d)
    tok, pos, grp, mask = e2.block_get()
    assert len(tok) == 128
    _, logits = e2.verify_forward(want_logits=True)
    cache = tf.KVCache(TINY); ob.prefill(W2, cache, list(prompt[:-1]))
    cands = [tok[8 + 15 * j: 8 + 15 * (j + 1)].tolist() for j in range(8)]
    t2, p2, g2, vis = ob.build_block(19, prompt[-1], d, cands)
    assert np.abs(logits.cpu().numpy() - tf.forward(W2, cache, t2, p2, vis)).max() < FP32_TOL
    eng.close(); e2.close()


# ----------------------------------------------- full-size verify step (the benchmark's configuration)

@pytest.mark.parametrize("L", [1024, 4096])
def test_verify_step_full_size_c2(L):
    """One 7B-shaped layer + LM head, 37-row candidate block on a random KV cache of L tokens, exactly as
    bench.py runs it: logits of every row against the oracle, acceptance and pool bit exact."""
    T, _, P, _ = synth.config("C2")
    w = synth.model_weights(T, 0, device="cuda:0")
    eng = binding.Engine(T, w, P)
    k, v = synth.kv_fill(T, 1, L, device="cuda:0")
    eng.tm.k_cache.copy_(k); eng.tm.v_cache.copy_(v)
    W = tf.Weights(T, {n: (t.cpu() if n != "layers" else [{a: b.cpu() for a, b in lw.items()} for lw in t]) for n, t in w.items()})
    cache = tf.KVCache(T, k.double().cpu().numpy(), v.double().cpu().numpy(), L)
    rng = np.random.default_rng(L)
    d = rng.integers(0, T.vocab, P.gamma).tolist()
    grams = np.concatenate([np.full((P.K, 1), d[-1]), rng.integers(0, T.vocab, (P.K, P.S))], axis=1)
    eng.phrase_update(grams)
    pool = oracle_pool(P)
    for g in grams:
        pool.insert(g)
    eng.set_state(L, 17)
    eng.assemble_candidates(draft=d)
    tok = eng.block_get()[0].tolist()
    tokens, pos, group, vis = ob.build_block(L, 17, d, pool.lookup(d[-1], P.K))
    assert tok == tokens and len(tok) == 37
    am, logits = eng.verify_forward(want_logits=True)
    want = tf.forward(W, cache, tokens, pos, vis)
    got = logits[:37].cpu().numpy().astype(np.float64)
    _bf16_tol(got, want)
    o = am[:37].cpu().numpy().tolist()
    n, chosen, A, acc = eng.accept_and_compact()
    A2, j2, m2, acc2 = ob.accept(tokens, o, P.gamma, P.S, P.K)
    assert (n, chosen, A, acc.tolist()) == (len(acc2), j2, A2, acc2)
    seq = [0] * L + [17] + acc2
    pool.apply(ob.harvest_ops(tokens, o, P.gamma, P.S, P.K, A2, seq, len(acc2), P))
    assert gpu_pool_rows(eng) == pool_rows(pool)
    eng.close()


# ------------------------------------------------------------ 7B-shaped pair: lossless at scale

def test_c3_shapes_ouroboros_is_bit_identical_to_vanilla():
    """Target 7B-shaped (32 layers), draft 1.1B-shaped (GQA 8:1, head_dim 64), bf16, replayed drafts and a
    replayed phrase source: the generated text must equal plain greedy decoding on the same kernels bit for
    bit, with phrase suffixes actually accepted along the way."""
    T, D, P, R = synth.config("C3")
    wt = synth.model_weights(T, 0, device="cuda:0")
    wd = synth.model_weights(D, 100, device="cuda:0")
    eng = binding.Engine(T, wt, P, D, wd)
    prompt = synth.prompt(0, T.vocab, 96, R["copy_frac"], *R["span"])
    gen = 72
    van, _ = eng.generate_vanilla(prompt, gen)
    truth = np.concatenate([prompt, van, np.zeros(64, dtype=np.int32)])

    def drafter(seq, g, step):
        d = synth.corrupt_drafts(5, truth, len(seq), g, T.vocab, 0.12, 0.03, step)
        grams = np.empty((P.K, P.beta), dtype=np.int32)
        for j in range(P.K):
            grams[j, 0] = d[-1]
            grams[j, 1:] = synth.corrupt_drafts(11 + j, truth, len(seq) + g, P.S, T.vocab, 0.08 * (j + 1), 0.0, step)
        eng.phrase_update(grams[::-1])
        return d

    eng.set_drafter(drafter)
    out, st = eng.generate(prompt, gen)
    eng.set_drafter(None)
    assert np.array_equal(out, van)
    assert st["suffix_tokens"] > 0 and st["target_calls"] < gen // 2
    nat, st2 = eng.generate(prompt, 24)                      # the draft model's own (chance-level) drafts
    assert np.array_equal(nat, van[:24]) and st2["draft_calls"] == 4 * st2["target_calls"]
    eng.close()


# ------------------------------------------------------------------- phrase-level drafting (Section 3.1)

def test_phrase_level_drafting_c1_matches_oracle():
    """The draft model drafts phrase by phrase: same text, same target calls and the oracle's number of draft
    forwards; against token-level drafting on the GPU only the number of draft forwards may differ."""
    import dataclasses
    P = dataclasses.replace(C1P, draft_phrases=True)
    w = synth.model_weights(C1T, 0, device="cuda:0")
    eng = binding.Engine(C1T, w, P, C1D, w)
    tok = binding.Engine(C1T, w, C1P, C1D, w)
    W = tf.Weights(C1T, synth.model_weights(C1T, 0))
    Wd = tf.Weights(C1D, synth.model_weights(C1T, 0))
    fewer = 0
    for seed in (0, 1, 4):
        prompt = synth.prompt(seed, C1T.vocab, C1R["n"], C1R["copy_frac"], *C1R["span"])
        gen = C1R["gen"]
        out, stats = eng.generate(prompt, gen)
        pool_gpu = gpu_pool_rows(eng)
        pool = oracle_pool(P)
        drafter = ob.PhraseDrafter(Wd, P, pool)
        trace = []
        ref, rstats = ob.generate(W, drafter, prompt, gen, P, pool=pool, trace=trace)
        assert out.tolist() == ref
        assert stats["target_calls"] == rstats["target_calls"] and stats["draft_calls"] == drafter.calls
        assert stats["suffix_tokens"] == sum(rstats["m"]) and stats["candidates"] == sum(rstats["n_cand"])
        assert pool_gpu[0] == [list(p) for _, p in trace[-1]["pool"]]
        out2, stats2 = tok.generate(prompt, gen)
        assert np.array_equal(out, out2) and stats2["target_calls"] == stats["target_calls"]
        assert stats2["draft_calls"] == P.gamma * stats2["target_calls"] >= stats["draft_calls"]
        fewer += stats2["draft_calls"] - stats["draft_calls"]
    assert fewer > 0                                   # some round did accept a phrase on the draft side
    eng.close()
    tok.close()


def test_phrase_level_drafting_bf16_self_draft():
    """bf16 on the tensor-core path, the target's own weights as the draft model: drafts are always accepted, the
    pool fills with the text's own phrases, and drafting by phrases must leave text and target calls untouched."""
    import dataclasses
    P0 = synth.DecodeParams(4, 9, 4, 32, 8)
    P1 = dataclasses.replace(P0, draft_phrases=True)
    w = synth.model_weights(MIDB, 3, device="cuda:0")
    prompt = synth.prompt(3, MIDB.vocab, 96, 0.3, 8, 32)
    res = []
    for P in (P0, P1):
        eng = binding.Engine(MIDB, w, P, MIDB, w)
        van, _ = eng.generate_vanilla(prompt, 120)
        out, st = eng.generate(prompt, 120)
        assert np.array_equal(out, van)
        res.append(st)
        eng.close()
    assert res[0]["target_calls"] == res[1]["target_calls"] and res[0]["full_accepts"] == res[0]["target_calls"]
    assert res[1]["draft_calls"] < res[0]["draft_calls"] == 4 * res[0]["target_calls"]     # c of Eq. 6 above 1


def test_phrase_level_drafting_edge_cases():
    """Long catch-up (the uncached text does not fit one block beside the candidates), K = 0 (every round is a plain
    single-token forward) and beta = 1 (phrases have no suffix): the drafts stay those of token-level drafting."""
    import dataclasses
    w = synth.model_weights(TINY, 2, device="cuda:0")
    prompt = synth.prompt(2, TINY.vocab, 125, 0.5, 4, 8)             # 125 + K*S rows > OURO_MAX_ROWS on the first round
    for gamma, beta, K in ((3, 4, 4), (3, 4, 0), (2, 1, 3)):
        P0 = synth.DecodeParams(gamma, beta, K, 8, 4)
        P1 = dataclasses.replace(P0, draft_phrases=True)
        outs = []
        for P in (P0, P1):
            eng = binding.Engine(TINY, w, P, TINY, w)
            van, _ = eng.generate_vanilla(prompt, 20)
            out, st = eng.generate(prompt, 20)
            assert np.array_equal(out, van)
            outs.append(st)
            eng.close()
        assert outs[0]["target_calls"] == outs[1]["target_calls"]
        assert outs[1]["draft_calls"] <= outs[0]["draft_calls"]
        if K == 0 or beta == 1:
            assert outs[1]["draft_calls"] == outs[0]["draft_calls"]


# --------------------------------------- tcgen05 attention: GQA, several rounds of query rows, span boundaries

GQAB = synth.ModelDesc(2, 512, 8, 2, 128, 1024, 1000, 1200, "bf16")   # 4 query heads per kv head, head_dim 128


def _gqa_case(P, seed, L_prompt):
    eng, W = make(GQAB, P, seed)
    rng = np.random.default_rng(seed)
    prompt = synth.prompt(seed, GQAB.vocab, L_prompt, 0.4, 4, 8)
    eng.reset()
    eng.prefill(prompt)
    d = rng.integers(0, GQAB.vocab, P.gamma).tolist()
    grams = rng.integers(0, GQAB.vocab, (P.K, P.beta)).astype(np.int32)
    grams[:, 0] = d[-1]
    eng.phrase_update(grams)
    pool = oracle_pool(P)
    for g in grams:
        pool.insert(g)
    eng.assemble_candidates(draft=d)
    tok = eng.block_get()[0]
    cands = pool.lookup(d[-1], P.K)
    t2, p2, g2, vis = ob.build_block(len(prompt) - 1, prompt[-1], d, cands)
    assert tok.tolist() == t2 and len(t2) == P.block_max
    am, logits = eng.verify_forward(want_logits=True)
    cache = tf.KVCache(GQAB)
    ob.prefill(W, cache, list(prompt[:-1]))
    want = tf.forward(W, cache, t2, p2, vis)
    got = logits[: len(t2)].cpu().numpy().astype(np.float64)
    _bf16_tol(got, want)
    err = np.abs(got - want).max(axis=1)
    srt = np.sort(want, axis=1)
    safe = (srt[:, -1] - srt[:, -2]) > 2 * err + 1e-12
    assert np.array_equal(am[: len(t2)].cpu().numpy()[safe], tf.argmax_rows(want)[safe])
    eng.close()


@pytest.mark.parametrize("seed,L_prompt", [(0, 40), (1, 509), (2, 1000), (3, 129)])
def test_verify_logits_bf16_gqa_head_dim_128(seed, L_prompt):
    """69 block rows x 4 query heads per kv head = 276 query rows (three rounds of 128) with 8 candidates, at
    cache lengths that put the block inside a chunk, across a span boundary (512) and at the end of a span."""
    _gqa_case(synth.DecodeParams(4, 9, 8, 16, 16, seed_prompt=False), seed, L_prompt)


@pytest.mark.parametrize("gamma,beta,K,L_prompt", [(7, 16, 8, 300), (3, 8, 16, 505)])
def test_verify_logits_bf16_widest_blocks(gamma, beta, K, L_prompt):
    """The widest block (128 rows: four rounds of query rows) and the most groups (16 candidates + trunk)."""
    _gqa_case(synth.DecodeParams(gamma, beta, K, 2, 32, seed_prompt=False), 5, L_prompt)


# ------------------------------------------------------------------ full-width shapes against the oracle

def _oracle_weights(desc, w):
    return tf.Weights(desc, {n: (t.cpu() if n != "layers" else [{a: b.cpu() for a, b in lw.items()} for lw in t]) for n, t in w.items()})


@pytest.mark.parametrize("name,K", [("C4", 8), ("C5", 4)])
def test_verify_logits_full_width_one_layer(name, K):
    """One decoder layer + LM head at the widths of the 34B- and 70B-shaped targets (d 7168 / 8192, 56 / 64 query
    heads on 8 kv heads, FFN 20480 / 28672, vocabulary 64000 / 32000): the candidate block (69 / 37 rows) on a
    prefilled cache, logits, greedy tokens and appended K/V against the oracle."""
    T, _, P, _ = synth.config(name)
    desc = dataclasses.replace(T, n_layers=1, max_seq=448)
    assert P.K == K and P.block_max == 1 + 4 + K * 8
    w = synth.model_weights(desc, 0, device="cuda:0")
    eng = binding.Engine(desc, w, P)
    W = _oracle_weights(desc, w)
    _verify_case(eng, W, desc, P, 2, 150, _bf16_tol, full_block=True)
    eng.close()


def test_teacher_forced_bf16_four_layer_7b_stack():
    """Four 7B-shaped layers (d 4096, FFN 11008, vocabulary 32000), bf16, ten decoding steps with replayed drafts and
    phrases: at every step the oracle evaluates the same block on the same history - logits within the bf16 bound,
    greedy tokens equal wherever the oracle's margin allows, acceptance / compaction / pool bit exact."""
    T, _, P, R = synth.config("C3")
    desc = dataclasses.replace(T, n_layers=4, max_seq=320)
    w = synth.model_weights(desc, 0, device="cuda:0")
    eng = binding.Engine(desc, w, P)
    W = _oracle_weights(desc, w)
    prompt = synth.prompt(1, desc.vocab, 48, R["copy_frac"], 4, 8)
    van, _ = eng.generate_vanilla(prompt, 96)
    truth = np.concatenate([prompt, van, np.zeros(64, dtype=np.int32)])
    eng.reset(); eng.prefill(prompt)
    cache = tf.KVCache(desc); ob.prefill(W, cache, list(prompt[:-1]))
    pool = oracle_pool(P); pool.apply(ob.prompt_ops(prompt, P.beta, P))
    seq = prompt.tolist()
    worst, suffix_tokens, full = 0.0, 0, 0
    for step in range(10):
        L = cache.length
        d = synth.corrupt_drafts(5, truth, len(seq), P.gamma, desc.vocab, 0.10, 0.03, step).tolist()
        grams = np.empty((P.K, P.beta), dtype=np.int32)
        for j in range(P.K):                                   # phrases that continue the draft, more or less corrupted
            grams[j, 0] = d[-1]
            grams[j, 1:] = synth.corrupt_drafts(11 + j, truth, len(seq) + P.gamma, P.S, desc.vocab, 0.08 * (j + 1), 0.0, step)
        eng.phrase_update(grams[::-1])
        for g in grams[::-1]:
            pool.insert(g)
        eng.assemble_candidates(draft=d)
        tok = eng.block_get()[0].tolist()
        cands = pool.lookup(d[-1], P.K)
        tokens, pos, group, vis = ob.build_block(L, seq[-1], d, cands)
        assert tok == tokens
        am, logits = eng.verify_forward(want_logits=True)
        want = tf.forward(W, cache, tokens, pos, vis)
        got = logits[: len(tokens)].cpu().numpy().astype(np.float64)
        rel = np.abs(got - want).max(axis=1) / np.abs(want).max(axis=1)
        worst = max(worst, rel.max())
        assert rel.max() < BF16_REL, (step, rel.max())
        err = np.abs(got - want).max(axis=1)
        srt = np.sort(want, axis=1)
        safe = (srt[:, -1] - srt[:, -2]) > 2 * err + 1e-12
        o = am[: len(tokens)].cpu().numpy()
        assert np.array_equal(o[safe], tf.argmax_rows(want)[safe])
        n, chosen, A, acc = eng.accept_and_compact()
        A2, j2, m2, acc2 = ob.accept(tokens, o.tolist(), P.gamma, P.S, len(cands))
        assert (n, chosen, A, acc.tolist()) == (len(acc2), j2, A2, acc2)
        ob.compact(cache, L, P.gamma, P.S, A2, j2, m2)
        seq += acc2
        pool.apply(ob.harvest_ops(tokens, o.tolist(), P.gamma, P.S, len(cands), A2, seq, len(acc2), P))
        assert gpu_pool_rows(eng) == pool_rows(pool)
        Ln = cache.length
        kv_tol = 2e-2 * max(np.abs(cache.k[:, :Ln]).max(), np.abs(cache.v[:, :Ln]).max())
        assert np.abs(eng.tm.k_cache[:, :Ln].float().cpu().numpy() - cache.k[:, :Ln]).max() < kv_tol
        assert np.abs(eng.tm.v_cache[:, :Ln].float().cpu().numpy() - cache.v[:, :Ln]).max() < kv_tol
        suffix_tokens += m2 if j2 >= 0 else 0
        full += A2 == P.gamma
        assert seq[len(prompt):] == van[: len(seq) - len(prompt)].tolist()      # the accepted text is the greedy text
    assert full >= 3 and suffix_tokens > 0, (full, suffix_tokens)
    eng.close()


@pytest.mark.parametrize("rows", [1, 37])
def test_exact_logit_ties_take_the_smallest_id(rows):
    """Identical rows of the LM head give bit-identical logits when they are accumulated the same way: inside one
    128-entry tile of the head GEMM, or in different tiles that one CTA handles over the whole K range (a tile whose
    K range is split across CTAs adds its partial sums in another order, so it rounds differently).  The greedy
    choice among such equals must be the smallest id - for a single row (plain decoding) and for a candidate block."""
    desc = synth.ModelDesc(1, 256, 4, 4, 64, 512, 32000, 192, "bf16")       # 250 head tiles: whole and split ones
    w = synth.model_weights(desc, 4, device="cuda:0")
    P = synth.DecodeParams(4, 9, 4, 16, 8, seed_prompt=False)
    eng = binding.Engine(desc, w, P)
    tokens = (np.arange(rows) * 7 + 3).astype(np.int32)
    eng.assemble_causal(binding.OURO_TARGET, tokens)
    _, lg = eng.verify_forward(want_logits=True)
    base = lg[:rows].clone()
    # a head row that wins for every token: a large multiple of the mean normalised activation direction is not
    # available from outside, so take the current winner's row of token 0 and scale it up
    win_id = int(base[0].argmax())
    boosted = (w["lm_head"][win_id].float() * 4.0).to(torch.bfloat16)
    # 250 tiles on 148 CTAs: tiles 0..147 are handled whole, 148..249 are split along K
    for ids in ((700, 731, 5000), (18900, 130, 131), (19050, 19000)):
        saved = {i: w["lm_head"][i].clone() for i in ids}
        for i in ids:
            w["lm_head"][i] = boosted
        am, lg = eng.verify_forward(want_logits=True)
        torch.cuda.synchronize()
        vals = {float(lg[0, i]) for i in ids}
        assert len(vals) == 1 and int(lg[0].argmax()) in ids, (vals, int(lg[0].argmax()))
        assert int(am[0]) == min(ids)
        for r in range(rows):                              # every row: the choice is the smallest index among the maxima
            mx = lg[r].max()
            assert int(am[r]) == int(torch.nonzero(lg[r] == mx)[0])
        am2, _ = eng.verify_forward()                      # and the same without materialised logits
        assert torch.equal(am2[:rows], am[:rows])
        for i in ids:
            w["lm_head"][i] = saved[i]
    eng.close()


# ------------------------------------------------------------------ a bounded device-side wait that runs out

def test_bounded_wait_gives_up_and_the_context_recovers():
    """The wait of a split-K tile for its other contributors is bounded.  With the bound set to zero polls it runs out
    at once (nothing is made to fault: the kernels return normally with the status word raised): the call that reads
    results back reports OURO_ETIMEOUT, plain decoding reports it too, and after a reset the same context computes
    oracle-equal logits again."""
    P = synth.DecodeParams(4, 9, 4, 16, 8)
    eng, W = make(MIDB, P, 2)                      # d 256: every q,k,v tile is split four ways
    _verify_case(eng, W, MIDB, P, 2, 40, _bf16_tol)
    eng.accept_and_compact()
    prompt = synth.prompt(2, MIDB.vocab, 40, 0.4, 4, 8)
    eng.set_wait_limit(0)
    eng.reset(); eng.prefill(prompt[:2])           # one causal row: raises the status word on the device
    eng.assemble_candidates(draft=[1, 2, 3, int(prompt[5])])
    eng.verify_forward()
    with pytest.raises(binding.OuroError) as e:
        eng.accept_and_compact()
    assert e.value.status == binding.OURO_ETIMEOUT
    with pytest.raises(binding.OuroError) as e:
        eng.generate_vanilla(prompt, 4)
    assert e.value.status == binding.OURO_ETIMEOUT
    eng.set_wait_limit(-1)
    _verify_case(eng, W, MIDB, P, 2, 40, _bf16_tol)     # reset + prefill + verify: as before the give-up
    eng.accept_and_compact()
    van, _ = eng.generate_vanilla(prompt, 12)
    eng.set_drafter(lambda seq, g, step: [int(van[min(len(seq) - len(prompt) + i, 11)]) for i in range(g)])
    out, _ = eng.generate(prompt, 12)
    eng.set_drafter(None)
    assert len(van) == 12 and np.array_equal(out, van)
    eng.close()


def test_tile_counter_generations_wrap_around(monkeypatch):
    """The split-K tile counters carry a generation number that grows with every GEMM; when the numbers are used up
    the words are cleared and counting starts over.  Started a few hundred GEMMs before that point, a generation
    crosses it and must still equal plain decoding token for token (which crosses it at another place)."""
    monkeypatch.setenv("OURO_GEN_START", str((1 << 22) - 300))
    P = synth.DecodeParams(4, 9, 4, 32, 8)
    eng, _ = make(MIDB, P, 5)
    prompt = synth.prompt(5, MIDB.vocab, 64, 0.3, 8, 32)
    van, _ = eng.generate_vanilla(prompt, 48)
    truth = np.concatenate([prompt, van, np.zeros(32, dtype=np.int32)])
    eng.set_drafter(lambda seq, g, step: synth.corrupt_drafts(1, truth, len(seq), g, MIDB.vocab, 0.1, 0.05, step))
    out, stats = eng.generate(prompt, 48)
    eng.set_drafter(None)
    assert np.array_equal(out, van) and stats["target_calls"] < 48
    eng.close()
    monkeypatch.delenv("OURO_GEN_START")
    eng2, _ = make(MIDB, P, 5)                       # and the same text from the usual starting point
    assert np.array_equal(eng2.generate_vanilla(prompt, 48)[0], van)
    eng2.close()


# ------------------------------------------------- phrase generation during the draft forward (Section 3.1)

def test_lookahead_window_matches_oracle_c1():
    """Every draft forward carries a lookahead window whose outputs refill it and feed the pool on the device: same text,
    target calls, accepted suffix tokens and pool as the oracle's LookaheadDrafter; candidates come up and get accepted
    without any phrase injected from outside."""
    P = dataclasses.replace(C1P, window=6)
    w = synth.model_weights(C1T, 0, device="cuda:0")
    W = tf.Weights(C1T, synth.model_weights(C1T, 0))
    for draft_desc in (C1D, C1T):                       # the early-exit draft, then the target as its own draft model
        eng = binding.Engine(C1T, w, P, draft_desc, w)
        Wd = tf.Weights(draft_desc, synth.model_weights(C1T, 0))
        got_suffix = got_cand = 0
        for seed in (1, 4):
            prompt = synth.prompt(seed, C1T.vocab, C1R["n"], C1R["copy_frac"], *C1R["span"])
            gen = C1R["gen"]
            out, stats = eng.generate(prompt, gen)
            pool_gpu = gpu_pool_rows(eng)
            van, _ = eng.generate_vanilla(prompt, gen)
            assert np.array_equal(out, van)
            pool = oracle_pool(P)
            drafter = ob.LookaheadDrafter(Wd, P, pool, P.window)
            trace = []
            ref, rstats = ob.generate(W, drafter, prompt, gen, P, pool=pool, trace=trace)
            assert out.tolist() == ref
            assert stats["target_calls"] == rstats["target_calls"] and stats["draft_calls"] == drafter.calls
            assert stats["suffix_tokens"] == sum(rstats["m"]) and stats["candidates"] == sum(rstats["n_cand"])
            assert pool_gpu[0] == [list(p) for _, p in trace[-1]["pool"]]
            got_suffix += stats["suffix_tokens"]
            got_cand += stats["candidates"]
        assert got_cand > 0
        if draft_desc is C1T:
            assert got_suffix > 0                       # the window's phrases are the target's own continuation
        eng.close()


def test_lookahead_window_bf16_self_draft():
    """The same on the tensor-core path (bf16, GQA, head dim 64): lossless, and the window's phrases extend accepted
    drafts although nothing but the prompt and the draft model's own forwards feeds the pool."""
    P0 = synth.DecodeParams(4, 9, 4, 32, 8)
    P1 = dataclasses.replace(P0, window=10)
    w = synth.model_weights(MIDB, 3, device="cuda:0")
    prompt = synth.prompt(3, MIDB.vocab, 96, 0.3, 8, 32)
    res = []
    for P in (P0, P1):
        eng = binding.Engine(MIDB, w, P, MIDB, w)
        van, _ = eng.generate_vanilla(prompt, 120)
        out, st = eng.generate(prompt, 120)
        assert np.array_equal(out, van)
        res.append(st)
        eng.close()
    assert res[1]["candidates"] > 0 and res[1]["suffix_tokens"] > 0
    assert res[1]["target_calls"] <= res[0]["target_calls"]
    with pytest.raises(binding.OuroError):              # a window together with phrase-level drafting is refused
        binding.Engine(MIDB, w, dataclasses.replace(P1, draft_phrases=True), MIDB, w)
