"""Pins for the procedure oracle: lossless invariant, packed == separate forwards, hand traces, properties."""
import json
import os

import numpy as np
import pytest

from oracle import ouroboros as ob
from oracle import transformer as tf
from paper_2402_13720_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")
TINY = synth.ModelDesc(2, 64, 4, 2, 16, 96, 100, 160, "f32")


def load_trace(name):
    out = {}
    for line in open(os.path.join(GOLD, name)):
        if line.strip() and not line.startswith("#"):
            k, v = line.split("=", 1)
            out[k.strip()] = json.loads(v)
    return out


def _params(gamma, beta, K, **kw):
    return synth.DecodeParams(gamma, beta, K, 8, 4, **kw)


# ------------------------------------------------------------------------------- hand traces

@pytest.mark.parametrize("name", ["trace_partial_accept.txt", "trace_full_accept.txt", "trace_tie.txt"])
def test_hand_traces(name):
    t = load_trace(name)
    gamma, beta = t["gamma"], t["beta"]
    S, L = beta - 1, 20
    tokens, pos, group, vis = ob.build_block(L, t["pending"], t["draft"], t["candidates"])
    if "positions_minus_L" in t:
        assert [p - L for p in pos] == t["positions_minus_L"]
    A, j, m, acc = ob.accept(tokens, t["outputs"], gamma, S, len(t["candidates"]))
    assert (A, j, m, acc) == (t["A"], t["chosen"], t["m"], t["accepted"])
    assert ob.n_match(tokens, t["outputs"], gamma) == t["n_match"] >= A
    desc = synth.ModelDesc(1, 8, 1, 1, 8, 8, 16, 64)
    cache = tf.KVCache(desc)
    cache.k[:] = np.arange(64)[None, :, None, None]
    cache.v[:] = -np.arange(64)[None, :, None, None]
    cache.length = L
    moves = ob.compact(cache, L, gamma, S, A, j, m)
    assert [[s - L, d - L] for s, d in moves] == t["moves"]
    assert cache.length - L == t["new_length_minus_L"] == len(acc)
    for s, d in moves:
        assert cache.k[0, d, 0, 0] == s and cache.v[0, d, 0, 0] == -s
    pure = dict(harvest_accepted=False, seed_prompt=False)
    if "ops_matched_only" in t:
        P = _params(gamma, beta, 0, harvest_candidates=False, **pure)
        ops = ob.harvest_ops(tokens, t["outputs"], gamma, S, 0, A, [], len(acc), P)
        assert [[o[0], list(o[1])] for o in ops] == t["ops_matched_only"]
        ops4 = ob.harvest_ops(tokens, t["outputs"], gamma, 3, 0, A, [], len(acc), _params(gamma, 4, 0, **pure))
        assert ops4 == t["ops_matched_only_beta4"]
    if "ops_candidates_only" in t:
        P = _params(gamma, beta, 2, harvest_matched=False, **pure)
        ops = ob.harvest_ops(tokens, t["outputs"], gamma, S, len(t["candidates"]), A, [], len(acc), P)
        assert [[o[0], list(o[1]), list(o[2])] for o in ops] == t["ops_candidates_only"]
        pool = ob.PhrasePool(8, 4, beta)
        for c in t["candidates"]:
            pool.insert([t["draft"][-1]] + c)
        pool.apply(ops)
        assert [list(p) for _, p in pool.export()] == t["pool_after"]


def test_hand_trace_harvest_accepted_windows():
    """Part 3 of harvest_ops (extension): which beta-windows of the text a step's accepted tokens yield."""
    t = load_trace("trace_harvest_accepted.txt")
    only = dict(harvest_matched=False, harvest_candidates=False, harvest_accepted=True, seed_prompt=False)

    def windows(seq, n_acc, beta):
        # block tokens / outputs are irrelevant with the other two parts switched off; A = 0 < gamma
        ops = ob.harvest_ops([0, 0], [0, 0], 1, beta - 1, 0, 0, seq, n_acc, _params(1, beta, 0, **only))
        assert all(op[0] == "insert" for op in ops)
        return [list(op[1]) for op in ops]

    for beta in (3, 4, 5, 6):
        assert windows(t["text_after"], t["n_accepted"], beta) == t[f"windows_beta{beta}"]
    assert windows(t["short_text_after"], t["short_n_accepted"], 3) == t["short_windows_beta3"]
    assert windows(t["single_text_after"], t["single_n_accepted"], 3) == t["single_windows_beta3"]
    off = dict(only, harvest_accepted=False)
    assert ob.harvest_ops([0, 0], [0, 0], 1, 2, 0, 0, t["text_after"], 2, _params(1, 3, 0, **off)) == []


def test_hand_trace_seed_prompt_windows():
    """prompt_ops (extension): every beta-window of the prompt, in order; none when the prompt is shorter."""
    t = load_trace("trace_seed_prompt.txt")
    for beta in (1, 3, 5, 6):
        ops = ob.prompt_ops(t["prompt"], beta, _params(2, beta, 1, seed_prompt=True))
        assert all(op[0] == "insert" for op in ops)
        assert [list(op[1]) for op in ops] == t[f"windows_beta{beta}"]
    assert ob.prompt_ops(t["prompt"], 3, _params(2, 3, 1, seed_prompt=False)) == []
    pool = ob.PhrasePool(1, 4, 3)
    pool.apply(ob.prompt_ops(t["prompt"], 3, _params(2, 3, 1)))
    assert [list(p) for _, p in pool.export()] == t["pool_after_beta3"]
    assert pool.lookup(1, 4) == t["lookup_1"] and pool.lookup(4, 4) == t["lookup_4"]


# -------------------------------------------------------------------- mask: packed == separate

@pytest.mark.parametrize("seed", [0, 1])
def test_packed_verification_equals_separate_causal_forwards(seed):
    """Eq. 8: the row that holds p^j_i must see exactly x, d_1..gamma, p^j_2..i.  So its logits equal those
    of a plain causal forward over that linear sequence, for each candidate separately."""
    W = tf.Weights(TINY, synth.model_weights(TINY, seed))
    rng = np.random.default_rng(seed)
    prefix = list(rng.integers(0, TINY.vocab, 13))
    gamma, S, K = 3, 4, 3
    d = list(rng.integers(0, TINY.vocab, gamma))
    cands = [list(rng.integers(0, TINY.vocab, S)) for _ in range(K)]
    cache = tf.KVCache(TINY)
    ob.prefill(W, cache, prefix[:-1])
    L = cache.length
    tokens, pos, group, vis = ob.build_block(L, prefix[-1], d, cands)
    packed = tf.forward(W, cache.clone(), tokens, pos, vis)
    for j in range(K):
        lin = prefix + d + cands[j]
        n = len(lin)
        ref = tf.forward(W, tf.KVCache(TINY), lin, list(range(n)), tf.causal_visible(0, n))
        assert np.abs(packed[: 1 + gamma] - ref[L:L + 1 + gamma]).max() < 1e-12
        rows = slice(1 + gamma + j * S, 1 + gamma + (j + 1) * S)
        assert np.abs(packed[rows] - ref[L + 1 + gamma:]).max() < 1e-12
    # a wrong mask (suffixes seeing each other causally) must fail this pin
    bad = tf.forward(W, cache.clone(), tokens, pos, tf.causal_visible(L, len(tokens)))
    assert np.abs(bad[-1] - packed[-1]).max() > 1e-6


def test_block_without_candidates_is_causal():
    tokens, pos, group, vis = ob.build_block(7, 1, [2, 3, 4], [])
    assert np.array_equal(vis, tf.causal_visible(7, 4)) and pos == [7, 8, 9, 10]


def test_mask_structure():
    L, gamma, S, K = 5, 2, 3, 2
    tokens, pos, group, vis = ob.build_block(L, 9, [1, 2], [[3, 4, 5], [6, 7, 8]])
    assert vis[:, :L].all()
    blk = vis[:, L:].astype(int)
    expect = np.array([
        [1, 0, 0, 0, 0, 0, 0, 0, 0],
        [1, 1, 0, 0, 0, 0, 0, 0, 0],
        [1, 1, 1, 0, 0, 0, 0, 0, 0],
        [1, 1, 1, 1, 0, 0, 0, 0, 0],
        [1, 1, 1, 1, 1, 0, 0, 0, 0],
        [1, 1, 1, 1, 1, 1, 0, 0, 0],
        [1, 1, 1, 0, 0, 0, 1, 0, 0],
        [1, 1, 1, 0, 0, 0, 1, 1, 0],
        [1, 1, 1, 0, 0, 0, 1, 1, 1]])
    assert np.array_equal(blk, expect)
    assert pos == [5, 6, 7, 8, 9, 10, 8, 9, 10]
    # a row's position equals the number of keys it sees minus one (it is a causal position)
    assert all(vis[r].sum() - 1 == pos[r] for r in range(len(pos)))


# ------------------------------------------------------------------------------ acceptance

def test_acceptance_properties_random():
    rng = np.random.default_rng(0)
    for _ in range(2000):
        gamma, S, K = int(rng.integers(1, 6)), int(rng.integers(1, 5)), int(rng.integers(0, 4))
        V = int(rng.integers(2, 4))                       # tiny vocabulary so matches are frequent
        B = 1 + gamma + K * S
        tokens, o = list(rng.integers(0, V, B)), list(rng.integers(0, V, B))
        A, j, m, acc = ob.accept(tokens, o, gamma, S, K)
        # Eq. 3
        assert 0 <= A <= gamma and all(tokens[1 + i] == o[i] for i in range(A))
        assert A == gamma or tokens[1 + A] != o[A]
        assert ob.n_match(tokens, o, gamma) >= A                     # Eq. 10
        assert 1 <= len(acc) <= gamma + S + 1
        if A < gamma or K == 0:
            assert j == -1 and acc == tokens[1:1 + A] + [o[A]]
        else:
            # Eq. 9 by brute force over every candidate and every possible accepted length
            ms = []
            for c in range(K):
                base = 1 + gamma + c * S
                chain = [o[gamma]] + [o[base + i] for i in range(S)]     # v^c_2 .. v^c_{beta+1}
                best = 0
                for a in range(1, S + 1):
                    if all(tokens[base + i] == chain[i] for i in range(a)):
                        best = a
                ms.append(best)
            assert m == max(ms) and j == ms.index(max(ms))
            base = 1 + gamma + j * S
            chain = [o[gamma]] + [o[base + i] for i in range(S)]
            assert acc == tokens[1:1 + gamma] + tokens[base:base + m] + [chain[m]]


# ------------------------------------------------------------------------------------ pool

def test_pool_policy_trace():
    """2 ways per set, everything in one set: insert order, refresh, eviction of the oldest, newest-first lookup."""
    p = ob.PhrasePool(1, 2, 3)
    p.insert((5, 1, 1)); p.insert((5, 2, 2))
    assert p.lookup(5, 4) == [[2, 2], [1, 1]]
    p.insert((5, 1, 1))                                  # refresh
    assert p.lookup(5, 4) == [[1, 1], [2, 2]] and p.lookup(5, 1) == [[1, 1]]
    p.insert((7, 3, 3))                                  # set full -> evicts the oldest, (5,2,2)
    assert p.lookup(5, 4) == [[1, 1]] and p.lookup(7, 4) == [[3, 3]] and p.lookup(6, 4) == []
    p.replace((5, 1, 1), (5, 9, 9))
    assert p.lookup(5, 4) == [[9, 9]]
    p.replace((5, 9, 9), (7, 3, 3))                      # verified version already present -> merged
    assert p.lookup(5, 4) == [] and [ph for _, ph in p.export()] == [(7, 3, 3)]
    assert p.clock == 6


def test_pool_lookup_postcondition_and_capacity():
    rng = np.random.default_rng(3)
    p = ob.PhrasePool(4, 3, 3)
    for _ in range(500):
        p.insert(tuple(rng.integers(0, 12, 3)))
        assert len(p.export()) <= 12
    for key in range(12):
        for suf in p.lookup(key, 3):
            assert (key, *suf) in [ph for _, ph in p.export()]
    assert ob.PhrasePool(128, 32, 4).set_of(1) == (2654435761 >> 25)


# ------------------------------------------------------------------- lossless, end to end

C1T, C1D, C1P, C1R = synth.config("C1")


@pytest.fixture(scope="module")
def c1():
    w = synth.model_weights(C1T, 0)
    return tf.Weights(C1T, w), tf.Weights(C1D, w)


def test_cached_greedy_equals_definition(c1):
    W, _ = c1
    prompt = synth.prompt(0, C1T.vocab, 12, 0.5, 4, 4)
    assert ob.vanilla_greedy(W, prompt, 10) == ob.greedy_definition(W, prompt, 10)


@pytest.mark.parametrize("seed,pure", [(0, False), (1, False), (2, True)])
def test_lossless_with_model_drafter(c1, seed, pure):
    """Eq. 4: whatever is drafted and whatever the pool holds, the accepted text is the target's own greedy text."""
    W, Wd = c1
    P = C1P.paper_pure() if pure else C1P
    prompt = synth.prompt(seed, C1T.vocab, C1R["n"], C1R["copy_frac"], *C1R["span"])
    ref = ob.vanilla_greedy(W, prompt, 40)
    trace = []
    out, stats = ob.generate(W, ob.ModelDrafter(Wd), prompt, 40, P, trace=trace)
    assert out == ref
    assert stats["target_calls"] <= 40 and 1.0 <= stats["eta"] <= P.gamma + P.beta
    assert all(1 <= n <= P.gamma + P.beta for n in stats["accepted"])
    for st in trace:                                       # the block is the trunk plus whole suffixes
        assert (len(st["tokens"]) - 1 - P.gamma) % P.S == 0 and len(st["tokens"]) <= P.block_max


@pytest.mark.parametrize("mode", ["self", "garbage", "replay"])
def test_lossless_with_other_drafters(c1, mode):
    W, _ = c1
    prompt = synth.prompt(5, C1T.vocab, 32, 0.5, 8, 8)
    ref = ob.vanilla_greedy(W, prompt, 48)
    if mode == "self":                                     # draft == target: the whole draft is always accepted
        drafter = ob.ModelDrafter(W)
    elif mode == "garbage":
        drafter = ob.FixedDrafter(lambda seq, g, step: [(7 * step + i) % C1T.vocab for i in range(g)])
    else:
        truth = np.array(list(prompt) + ref + [0] * 16)
        drafter = ob.FixedDrafter(lambda seq, g, step: synth.corrupt_drafts(9, truth, len(seq), g, C1T.vocab, 0.1, 0.1, step))
    out, stats = ob.generate(W, drafter, prompt, 48, C1P)
    assert out == ref
    if mode == "self":
        assert all(a == C1P.gamma for a in stats["A"])
    if mode == "garbage":
        assert max(stats["A"]) <= 1
    if mode == "replay":
        assert stats["eta"] > 1.5 and max(stats["m"]) >= 1      # phrases do extend accepted drafts


def test_eta_is_one_when_nothing_is_accepted(c1):
    W, _ = c1
    prompt = synth.prompt(6, C1T.vocab, 16, 0.0, 8, 8)
    ref = ob.vanilla_greedy(W, prompt, 12)
    wrong = ob.FixedDrafter(lambda seq, g, step: [(ref[min(len(seq) - 16, 11)] + 1) % C1T.vocab] * g)
    out, stats = ob.generate(W, wrong, prompt, 12, C1P.paper_pure())
    assert out == ref and stats["eta"] == 1.0 and stats["target_calls"] == 12


def test_compaction_equals_fresh_prefill(c1):
    """After every step the cache must hold exactly the K/V of the accepted text."""
    W, _ = c1
    prompt = synth.prompt(9, C1T.vocab, 32, 0.5, 8, 8)
    ref = ob.vanilla_greedy(W, prompt, 64)
    truth = np.array(list(prompt) + ref + [0] * 16)
    drafter = ob.FixedDrafter(lambda seq, g, step: synth.corrupt_drafts(3, truth, len(seq), g, C1T.vocab, 0.05, 0.05, step))
    P = C1P
    pool = ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)
    pool.apply(ob.prompt_ops(prompt, P.beta, P))
    cache = tf.KVCache(C1T)
    ob.prefill(W, cache, list(prompt[:-1]))
    seq, moved = [int(t) for t in prompt], 0
    for step in range(11):
        L = cache.length
        d = drafter.draft(seq, P.gamma, step)
        cands = pool.lookup(d[-1], P.K)
        tokens, pos, group, vis = ob.build_block(L, seq[L], d, cands)
        o = tf.argmax_rows(tf.forward(W, cache, tokens, pos, vis))
        A, j, m, acc = ob.accept(tokens, o, P.gamma, P.S, len(cands))
        moved += len(ob.compact(cache, L, P.gamma, P.S, A, j, m))
        seq += acc
        pool.apply(ob.harvest_ops(tokens, o, P.gamma, P.S, len(cands), A, seq, len(acc), P))
        fresh = tf.KVCache(C1T)
        ob.prefill(W, fresh, seq[:-1])
        assert cache.length == fresh.length == len(seq) - 1
        assert np.abs(cache.k[:, :cache.length] - fresh.k[:, :fresh.length]).max() < 1e-12
        assert np.abs(cache.v[:, :cache.length] - fresh.v[:, :fresh.length]).max() < 1e-12
    assert moved > 0          # the scenario did exercise a real move


def test_history_reuse_keeps_losslessness(c1):
    """Section 3.4: a pool carried over from an earlier query changes speed, never the text."""
    W, Wd = c1
    pool = ob.PhrasePool(C1P.pool_sets, C1P.pool_ways, C1P.beta)
    for seed in (10, 11):
        prompt = synth.prompt(seed, C1T.vocab, 24, 0.5, 8, 8)
        out, _ = ob.generate(W, ob.ModelDrafter(Wd), prompt, 24, C1P, pool=pool)
        assert out == ob.vanilla_greedy(W, prompt, 24)
    assert len(pool.export()) > 0


def test_eos_stops_generation(c1):
    W, Wd = c1
    prompt = synth.prompt(0, C1T.vocab, 32, 0.5, 8, 8)
    ref = ob.vanilla_greedy(W, prompt, 30)
    eos = ref[9]
    cut = ref[: ref.index(eos) + 1]
    import dataclasses
    P = dataclasses.replace(C1P, eos_token=eos)
    out, _ = ob.generate(W, ob.ModelDrafter(Wd), prompt, 30, P)
    assert out == cut == ob.vanilla_greedy(W, prompt, 30, eos=eos)


# ------------------------------------------------------------------- phrase-level drafting (Section 3.1)

class _Spy:
    """Runs two drafters side by side on the same calls and records what each returned."""

    def __init__(self, a, b):
        self.a, self.b, self.log = a, b, []

    def draft(self, seq, gamma, step):
        da, db = self.a.draft(seq, gamma, step), self.b.draft(seq, gamma, step)
        self.log.append((da, db))
        return da

    def rollback(self, valid_len):
        self.a.rollback(valid_len)
        self.b.rollback(valid_len)


@pytest.mark.parametrize("seed", [0, 3])
def test_phrase_drafter_gives_the_token_level_drafts(c1, seed):
    """Eq. 4 applied to the draft model: drafting by phrases changes how many forwards the draft model runs,
    never what it drafts.  The token-level drafter (Eq. 1) is the independent definition."""
    W, Wd = c1
    prompt = synth.prompt(seed, C1T.vocab, C1R["n"], C1R["copy_frac"], *C1R["span"])
    pool = ob.PhrasePool(C1P.pool_sets, C1P.pool_ways, C1P.beta)
    tok, phr = ob.ModelDrafter(Wd), ob.PhraseDrafter(Wd, C1P, pool)
    spy = _Spy(tok, phr)
    out, stats = ob.generate(W, spy, prompt, 40, C1P, pool=pool)
    assert out == ob.vanilla_greedy(W, prompt, 40)
    assert all(a == b and len(b) == C1P.gamma for a, b in spy.log)
    assert phr.calls <= C1P.gamma * stats["target_calls"]
    assert tok.cache.length >= phr.cache.length - 1           # the phrase drafter may also hold d_gamma


def test_phrase_drafter_saves_forwards_when_the_pool_knows_the_continuation(c1):
    """A pool phrase equal to the draft model's own greedy continuation is accepted whole: one forward yields
    1 + S tokens (c of Eq. 6 above 1); a pool of wrong phrases costs nothing but yields one token per forward."""
    W, Wd = c1
    P = C1P
    prompt = [int(t) for t in synth.prompt(5, C1T.vocab, 20, 0.0, 4, 4)]
    cont = ob.vanilla_greedy(Wd, prompt, P.gamma + 2)          # the draft model's own greedy text
    good = ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)
    good.insert([prompt[-1]] + cont[:P.S])
    d = ob.PhraseDrafter(Wd, P, good)
    assert d.draft(prompt, P.gamma, 0) == cont[:P.gamma]
    assert d.calls == -(-P.gamma // (P.S + 1))                # ceil(gamma / (1 + S)) rounds
    bad = ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)
    bad.insert([prompt[-1]] + [(cont[0] + 1) % C1T.vocab] * P.S)
    d2 = ob.PhraseDrafter(Wd, P, bad)
    assert d2.draft(prompt, P.gamma, 0) == cont[:P.gamma] and d2.calls == P.gamma


def test_phrase_drafter_cache_equals_fresh_prefill(c1):
    """After rounds that accepted phrase suffixes the draft cache holds exactly the K/V of its text."""
    W, Wd = c1
    P = C1P
    prompt = [int(t) for t in synth.prompt(6, C1T.vocab, 20, 0.0, 4, 4)]
    cont = ob.vanilla_greedy(Wd, prompt, 8)
    pool = ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)
    pool.insert([prompt[-1]] + [(cont[0] + 1) % C1T.vocab] * P.S)      # tried first (newest last -> insert order below)
    pool.insert([prompt[-1]] + cont[:P.S])
    pool.insert([prompt[-1]] + [(cont[0] + 2) % C1T.vocab] * P.S)      # newest: candidate 0, wrong; the good one is candidate 1
    d = ob.PhraseDrafter(Wd, P, pool)
    out = d.draft(prompt, P.gamma, 0)
    assert out == cont[:P.gamma]
    text = prompt + out
    n = d.cache.length
    fresh = tf.KVCache(C1D)
    tf.forward(Wd, fresh, text[:n], list(range(n)), tf.causal_visible(0, n))
    assert n >= len(prompt) + P.S and np.abs(d.cache.k[:, :n] - fresh.k[:, :n]).max() < 1e-12
    assert np.abs(d.cache.v[:, :n] - fresh.v[:, :n]).max() < 1e-12


def test_draft_accept_planted_mistake():
    """Chain of Eq. 9 on the draft side: the first suffix token is checked against o[n-1], not against o[n]."""
    S, n = 3, 2
    tokens = [7, 8, 20, 21, 22, 20, 30, 31]                  # trunk 7 8; candidates (20 21 22), (20 30 31)
    o = [0, 20, 21, 99, 0, 30, 31, 55]                       # after 8 comes 20; cand 0 matches 2, cand 1 matches 3
    assert ob.draft_accept(tokens, o, n, S, 2) == (1, 3, [20, 30, 31, 55])
    assert ob.draft_accept(tokens, o, n, S, 1) == (0, 2, [20, 21, 99])
    assert ob.draft_accept(tokens, o, n, S, 0) == (-1, 0, [20])


# ------------------------------------------------- phrase generation during the draft forward (Section 3.1)

def test_hand_trace_window_phrases():
    t = load_trace("trace_window_phrases.txt")
    for beta in (3, 4, 5, 6, 7):
        got = ob.window_phrases(t["src"], t["chain"], beta - 1)
        assert [list(p) for p in got] == t[f"phrases_beta{beta}"]
    assert t["chain"][1:] == t["next_window"]


def test_lookahead_window_fixed_point_and_drafts(c1):
    """Jacobi fixed point: a window that already holds the draft model's own greedy continuation is reproduced by the
    forward (each window row then sees exactly the true text), which pins the window rows' positions and mask against
    plain causal decoding; a wrong mask (window rows not seeing each other) fails it.  The drafts themselves are those
    of the plain token-level drafter whatever the window holds."""
    W, Wd = c1
    P = C1P
    width = 6
    prompt = [int(t) for t in synth.prompt(7, C1T.vocab, 20, 0.0, 4, 4)]
    cont = ob.vanilla_greedy(Wd, prompt, P.gamma + width + 2)            # the draft model's own greedy text
    pool = ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)
    d = ob.LookaheadDrafter(Wd, P, pool, width)
    d.window = cont[:width]                                              # exact guesses for the positions after the prompt
    out = d.draft(prompt, 1, 0)
    assert out == cont[:1] and d.window == cont[1:1 + width]             # reproduced and slid by one
    bad = ob.LookaheadDrafter(Wd, P, ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta), width)
    bad.window = cont[:width]
    import unittest.mock as um
    real_block = ob.build_block

    def wrong_mask(L, pending, draft, cands):                            # window rows that do not see one another
        tokens, pos, group, vis = real_block(L, pending, draft, cands)
        n = 1 + len(draft)
        for r in range(n, len(tokens)):
            vis[r, L + n:L + r] = False
        return tokens, pos, group, vis

    with um.patch.object(ob, "build_block", wrong_mask):
        bad.draft(prompt, 1, 0)
    assert bad.window != cont[1:1 + width]
    # every phrase of that forward is then exact greedy text of the draft model
    text = prompt + cont
    for _, ph in pool.export():
        k = [i for i in range(len(prompt) - 1, len(text) - P.beta + 1) if tuple(text[i:i + P.beta]) == ph]
        assert k, ph
    # garbage guesses: the drafts are still those of plain drafting (the real rows never see the window)
    d2 = ob.LookaheadDrafter(Wd, P, ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta), width)
    d2.window = [(cont[i] + 1) % C1T.vocab for i in range(width)]
    assert d2.draft(prompt, P.gamma, 0) == ob.ModelDrafter(Wd).draft(prompt, P.gamma, 0) == cont[:P.gamma]
    # width 0: nothing but plain drafting, the pool is not touched
    p0 = ob.PhrasePool(P.pool_sets, P.pool_ways, P.beta)
    d0 = ob.LookaheadDrafter(Wd, P, p0, 0)
    assert d0.draft(prompt, P.gamma, 0) == cont[:P.gamma] and p0.export() == []


@pytest.mark.parametrize("seed", [0, 4])
def test_lossless_with_lookahead_drafter(c1, seed):
    """Phrases made during drafting change what is verified, never the text (Eq. 4); with the target's own weights as
    the draft model the window's phrases are the target's continuation and get accepted."""
    W, Wd = c1
    prompt = synth.prompt(seed, C1T.vocab, C1R["n"], C1R["copy_frac"], *C1R["span"])
    ref = ob.vanilla_greedy(W, prompt, 40)
    for draft_w in (Wd, W):
        pool = ob.PhrasePool(C1P.pool_sets, C1P.pool_ways, C1P.beta)
        out, stats = ob.generate(W, ob.LookaheadDrafter(draft_w, C1P, pool, 6), prompt, 40, C1P, pool=pool)
        assert out == ref
    assert sum(stats["m"]) > 0 and sum(stats["n_cand"]) > 0       # self-draft: suffixes from the window's phrases accepted
