"""CPU oracle, part 2: the Ouroboros decoding procedure around the verification forward.

TEST INFRASTRUCTURE ONLY.  Plain Python over lists, one function per step of the method, in the
paper's order and notation.  Shares no code with the CUDA path.

Notation (Section 2 and Section 3.2): the prefix is x; the last accepted token, whose K/V is not
cached yet, is the *pending* token and occupies block row 0; d_1..d_gamma is the draft; a phrase
p_1..p_beta starts with p_1 = d_gamma, so a candidate contributes S = beta - 1 suffix rows; o_b is
the target's greedy next-token choice at block row b.

What the paper fixes and what is this build's reading:
  * Eq. 1-4 (draft, verify, accurate prefix A, equivalence to autoregressive decoding), Eq. 7-9
    (K lengthened drafts, per-suffix conditionals, suffix acceptance) are followed as printed.
    The printed range "j = 2..K" under Eq. 7 is read as j = 1..K.
  * Ties for "the phrase with the largest accepted suffix" go to the earliest candidate.
  * The phrase pool's layout, capacity, eviction and ordering are not given by the paper: a
    sets x ways table addressed by the first token, LRU by a global stamp (PhrasePool below).
  * Phrase-level drafting on the draft model (Section 3.1) is not specified by the paper; PhraseDrafter
    is this build's reading: the draft model verifies pool phrases on itself, Section 3.2 style.
  * Phrase generation during the draft forward (Section 3.1 defers to lookahead decoding) is not specified
    either; LookaheadDrafter / window_phrases is this build's reading: a sliding window of guessed tokens
    rides along every draft forward, one Jacobi step per forward, and its diagonals are the new phrases.
  * "Sub-segments of the discarded draft that match the verification" (Section 3.3) is read as
    in harvest_ops(); the replacement of tried phrases by their verified versions follows the
    second paragraph of Section 3.3.

Pins (tests/test_oracle_ouroboros.py): generated tokens equal plain greedy decoding from the
definition (Eq. 4) for every seed and flag setting; packed verification equals K separate
causal forwards (Eq. 8); hand traces under tests/golden/; Eq. 3 / Eq. 9 / Eq. 10 properties;
compaction equals a fresh prefill.  The pool policy and the harvest readings are this build's
(the paper is silent); each is fixed by a hand-worked trace: the pool by its policy trace, the matched
sub-segments and tried phrases by the three step traces, the two extensions (windows of the accepted
text, windows of the prompt) by trace_harvest_accepted.txt and trace_seed_prompt.txt, the lookahead window's
phrases by trace_window_phrases.txt; its block (positions, mask) by the Jacobi fixed point: a window that
already holds the draft model's greedy continuation reproduces it.
"""
from __future__ import annotations

import numpy as np

from . import transformer as tf


# ----------------------------------------------------------------------------------- phrase pool

class PhrasePool:
    """sets x ways table of beta-grams keyed by their first token, newest-first retrieval.

    set(key) = ((key * 2654435761) mod 2^32) >> (32 - log2(sets)).  Every insert or refresh
    takes the next value of a global counter as the entry's stamp."""

    def __init__(self, sets, ways, beta):
        assert sets & (sets - 1) == 0
        self.sets, self.ways, self.beta = sets, ways, beta
        self.entries = [[None] * ways for _ in range(sets)]   # None or [phrase tuple, stamp]
        self.clock = 0

    def set_of(self, key):
        bits = self.sets.bit_length() - 1
        return ((key * 2654435761) & 0xFFFFFFFF) >> (32 - bits) if bits else 0

    def _find(self, phrase):
        row = self.entries[self.set_of(phrase[0])]
        for w, e in enumerate(row):
            if e is not None and e[0] == phrase:
                return row, w
        return row, None

    def insert(self, phrase):
        """Present: refresh its stamp.  Else first free way.  Else overwrite the oldest stamp in the set."""
        phrase = tuple(int(t) for t in phrase)
        assert len(phrase) == self.beta
        self.clock += 1
        row, w = self._find(phrase)
        if w is None:
            free = [i for i, e in enumerate(row) if e is None]
            w = free[0] if free else min(range(self.ways), key=lambda i: row[i][1])
        row[w] = [phrase, self.clock]

    def erase(self, phrase):
        row, w = self._find(tuple(int(t) for t in phrase))
        if w is not None:
            row[w] = None

    def replace(self, old, new):
        """The tried phrase ``old`` becomes its verified version ``new`` (Section 3.3): equal -> refresh;
        otherwise ``old`` leaves the pool and ``new`` enters by the insert rule (merging with a duplicate)."""
        if tuple(old) != tuple(new):
            self.erase(old)
        self.insert(new)

    def lookup(self, key, K):
        """Up to K suffixes p_2..p_beta of the phrases with p_1 = key, most recent first (Section 3.2)."""
        hits = [e for e in self.entries[self.set_of(key)] if e is not None and e[0][0] == key]
        hits.sort(key=lambda e: -e[1])
        return [list(e[0][1:]) for e in hits[:K]]

    def export(self):
        """All phrases with their stamps, oldest first."""
        flat = [(e[1], e[0]) for row in self.entries for e in row if e is not None]
        return sorted(flat)

    def apply(self, ops):
        for op in ops:
            if op[0] == "insert":
                self.insert(op[1])
            else:
                self.replace(op[1], op[2])


# ----------------------------------------------------------------------------- block and mask

def build_block(L, pending, draft, cands):
    """Pack the K lengthened drafts of Eq. 7 into one query block.

    Rows: 0 = pending token, 1..gamma = d_1..d_gamma (the trunk), then candidate j's suffix
    p^j_2..p^j_beta at rows 1+gamma+j*S+(i-1), i = 1..S.  Position of a trunk row b is L+b; of
    suffix row (j, i) it is L+gamma+i.  Visibility (Eq. 8): every row sees the whole cache; trunk
    row b sees trunk rows <= b; suffix row (j, i) sees the whole trunk and rows (j, 1..i) only."""
    gamma, Kc = len(draft), len(cands)
    S = len(cands[0]) if Kc else 0
    tokens = [int(pending)] + [int(t) for t in draft] + [int(t) for c in cands for t in c]
    B = len(tokens)
    pos = [L + b for b in range(1 + gamma)] + [L + gamma + i for _ in range(Kc) for i in range(1, S + 1)]
    group = [0] * (1 + gamma) + [1 + j for j in range(Kc) for _ in range(S)]
    visible = np.zeros((B, L + B), dtype=bool)
    visible[:, :L] = True
    for r in range(B):
        for c in range(B):
            if group[c] == 0:
                visible[r, L + c] = c <= r if group[r] == 0 else True
            else:
                visible[r, L + c] = group[c] == group[r] and c <= r
    return tokens, pos, group, visible


# ------------------------------------------------------------------------------------ acceptance

def accept(tokens, o, gamma, S, n_cand):
    """Greedy acceptance.  Returns (A, j_star, m, accepted).

    A (Eq. 3): the largest a with d_1..a = v_1..a, where v_i = o_{i-1}.  If A < gamma the step
    accepts d_1..A and v_{A+1} (Section 2).  If A = gamma, candidate j's verified chain is
    v^j_2 = o_gamma, v^j_{i+1} = o at suffix row (j, i-1); m_j = hat-A^j - 1 is the number of its
    suffix tokens matching that chain (Eq. 9); the candidate with the largest m_j wins (earliest
    on ties) and the step accepts d, its m_j matched tokens and the chain's next token."""
    A = 0
    while A < gamma and tokens[1 + A] == o[A]:
        A += 1
    if A < gamma or n_cand == 0:
        return A, -1, 0, [int(t) for t in tokens[1:1 + A]] + [int(o[A])]
    best = (-1, -1, None)
    for j in range(n_cand):
        base, m, v = 1 + gamma + j * S, 0, o[gamma]
        while m < S and tokens[base + m] == v:
            v = o[base + m]
            m += 1
        if m > best[1]:
            best = (j, m, v)
    j, m, v = best
    base = 1 + gamma + j * S
    return A, j, m, [int(t) for t in tokens[1:1 + gamma]] + [int(t) for t in tokens[base:base + m]] + [int(v)]


def n_match(tokens, o, gamma):
    """#Match of Eq. 10: how many draft tokens equal the verification result at their position."""
    return sum(1 for i in range(1, gamma + 1) if tokens[i] == o[i - 1])


def compact(cache, L, gamma, S, A, j, m):
    """Keep slots L..L+A (pending token and accepted draft); if a suffix was accepted move its m slots
    next to the trunk.  Rejected rows are simply left beyond the new length.  Returns the (src, dst) moves."""
    moves = []
    if j >= 0 and m > 0:
        src0, dst0 = L + 1 + gamma + j * S, L + 1 + gamma
        for t in range(m):
            if src0 != dst0:
                cache.k[:, dst0 + t], cache.v[:, dst0 + t] = cache.k[:, src0 + t].copy(), cache.v[:, src0 + t].copy()
                moves.append((src0 + t, dst0 + t))
    cache.length = L + 1 + A + (m if j >= 0 else 0)
    return moves


# --------------------------------------------------------------------------------------- harvest

def harvest_ops(tokens, o, gamma, S, n_cand, A, seq_after, n_acc, P):
    """Pool updates after one verification, as an ordered list of operations.

    1. Tried phrases (Section 3.3, second paragraph), only when the draft was fully accepted:
       every candidate j, in order, is replaced by (d_gamma, v^j_2, .., v^j_beta), the target's own
       continuation under that candidate's context.  For the chosen candidate this is the same rule
       (a fully matched phrase equals its verified version and is merely refreshed).
    2. Matched sub-segments of the discarded draft (Section 3.3, first paragraph), only when A < gamma:
       for every trunk row s whose token lies in the discarded region (A+1 <= s <= gamma-1), if the
       following draft tokens agree with the target's outputs (t_{s+q} = o_{s+q-1}) for q = 1..beta-2
       at least, the beta-gram (t_s, o_s, .., o_{s+beta-2}) is inserted: its first token is the key and
       every later token is a target prediction.  A run must have at least one match; shorter chains
       are dropped because the pool holds beta-grams only.
    3. Extension (not in the paper): every beta-window of the running text that ends inside the newly
       accepted tokens."""
    beta, ops = S + 1, []
    if P.harvest_candidates and A == gamma and n_cand > 0:
        for j in range(n_cand):
            base = 1 + gamma + j * S
            old = [tokens[gamma]] + list(tokens[base:base + S])
            new = [tokens[gamma], o[gamma]] + [o[base + i] for i in range(S - 1)]
            ops.append(("replace", tuple(int(t) for t in old), tuple(int(t) for t in new)))
    if P.harvest_matched and A < gamma:
        for s in range(A + 1, gamma):
            r = 0
            while s + r + 1 <= gamma and tokens[s + r + 1] == o[s + r]:
                r += 1
            if r >= max(1, beta - 2):
                ops.append(("insert", tuple([int(tokens[s])] + [int(o[s + q]) for q in range(beta - 1)])))
    if P.harvest_accepted:
        n = len(seq_after)
        for e in range(n - n_acc, n):
            if e - beta + 1 >= 0:
                ops.append(("insert", tuple(int(t) for t in seq_after[e - beta + 1:e + 1])))
    return ops


def prompt_ops(prompt, beta, P):
    """Extension (not in the paper): seed the pool with every beta-window of the prompt."""
    if not P.seed_prompt:
        return []
    return [("insert", tuple(int(t) for t in prompt[i:i + beta])) for i in range(len(prompt) - beta + 1)]


# ------------------------------------------------------------------------------------- decoding

def greedy_definition(W, prompt, max_new):
    """Autoregressive greedy decoding exactly as defined: every new token is the argmax of a full
    causal forward over the whole sequence so far (no cache, no block tricks)."""
    seq = [int(t) for t in prompt]
    for _ in range(max_new):
        n = len(seq)
        cache = tf.KVCache(W.desc)
        logits = tf.forward(W, cache, seq, list(range(n)), tf.causal_visible(0, n))
        seq.append(int(tf.argmax_rows(logits[-1:])[0]))
    return seq[len(prompt):]


def prefill(W, cache, tokens):
    """Cache every given token with one causal forward (the pending token is not part of ``tokens``)."""
    n = len(tokens)
    if n:
        tf.forward(W, cache, tokens, list(range(cache.length, cache.length + n)), tf.causal_visible(cache.length, n))
        cache.length += n


def vanilla_greedy(W, prompt, max_new, eos=-1):
    """Greedy decoding with a KV cache, one target forward per token (the timed baseline of Section 4.1)."""
    cache = tf.KVCache(W.desc)
    prefill(W, cache, list(prompt[:-1]))
    pending, out = int(prompt[-1]), []
    while len(out) < max_new:
        L = cache.length
        logits = tf.forward(W, cache, [pending], [L], tf.causal_visible(L, 1))
        cache.length = L + 1
        pending = int(tf.argmax_rows(logits)[0])
        out.append(pending)
        if pending == eos:
            break
    return out


class ModelDrafter:
    """Token-level greedy drafting with the draft model (Eq. 1); keeps its own cache of the text."""

    def __init__(self, W):
        self.W, self.cache = W, tf.KVCache(W.desc)

    def draft(self, seq, gamma, step):
        """seq = whole text including the pending token.  Returns d_1..d_gamma."""
        c, out = self.cache, []
        feed = [int(t) for t in seq[c.length:]]
        for _ in range(gamma):
            n, L = len(feed), c.length
            logits = tf.forward(self.W, c, feed, list(range(L, L + n)), tf.causal_visible(L, n))
            c.length = L + n
            feed = [int(tf.argmax_rows(logits[-1:])[0])]
            out.append(feed[0])
        return out

    def rollback(self, valid_len):
        self.cache.length = min(self.cache.length, valid_len)


def draft_accept(tokens, o, n, S, n_cand):
    """One phrase-level drafting round of the draft model.  Rows 0..n-1 of the block are text the draft
    model is being fed (nothing to verify there), so its next greedy token is o[n-1]; candidate j's
    chain continues from it exactly as in Eq. 9.  Returns (j_star, m, gained): the chosen candidate
    (-1 without candidates), its matched suffix tokens, and the 1 + m tokens the round yields."""
    if n_cand == 0:
        return -1, 0, [int(o[n - 1])]
    best = (-1, -1, None)
    for j in range(n_cand):
        base, m, v = n + j * S, 0, o[n - 1]
        while m < S and tokens[base + m] == v:
            v = o[base + m]
            m += 1
        if m > best[1]:
            best = (j, m, v)
    j, m, v = best
    return j, m, [int(t) for t in tokens[n + j * S:n + j * S + m]] + [int(v)]


class PhraseDrafter:
    """Phrase-level drafting on the draft model (Section 3.1, Eq. 6: gamma draft tokens for gamma / c
    draft forwards).  The paper gives no procedure ("we will not go into detail ..."), so this is this
    build's reading: a drafting round is the verification step of Section 3.2 run by the DRAFT model on
    itself.  The round's block is the text the draft model has not cached yet followed by the K pool
    phrases that start with the last known token, under the mask of Eq. 8; the draft model's greedy
    outputs accept the longest matching phrase prefix (Eq. 9) plus one more token.  The drafts are, by
    Eq. 4 applied to the draft model, the ones token-level drafting (Eq. 1) would produce; only the
    number of draft forwards changes.  The pool is read, never written, while drafting."""

    def __init__(self, W, P, pool):
        self.W, self.P, self.pool, self.cache = W, P, pool, tf.KVCache(W.desc)
        self.calls = 0

    def draft(self, seq, gamma, step):
        c, S, out = self.cache, self.P.S, []
        feed = [int(t) for t in seq[c.length:]]
        while len(out) < gamma:
            n, L = len(feed), c.length
            cands = self.pool.lookup(feed[-1], self.P.K) if S > 0 else []
            tokens, pos, group, visible = build_block(L, feed[0], feed[1:], cands)
            o = tf.argmax_rows(tf.forward(self.W, c, tokens, pos, visible))
            self.calls += 1
            j, m, gained = draft_accept(tokens, o, n, S, len(cands))
            keep = min(len(gained), gamma - len(out))       # a draft has exactly gamma tokens
            mk = min(m, keep)                                # kept tokens whose K/V the round computed
            compact(c, L, n - 1, S, n - 1, j, mk)
            c.length = L + n + mk
            out += gained[:keep]
            feed = [out[-1]]
        return out

    def rollback(self, valid_len):
        self.cache.length = min(self.cache.length, valid_len)


def window_phrases(src, chain, S):
    """Phrases one draft forward with a lookahead window yields (this build's reading of Section 3.1's "multiple new
    phrases are generated in parallel during each forward of the draft model"; the paper gives no procedure).

    src[0] is the last real token the forward was fed and src[1..W] the window's guesses for the positions after
    it; chain[i] is the draft model's greedy output at the row that holds src[i], i.e. its prediction for the next
    position given the real text and the guesses src[1..i].  Along the diagonal, src[i] followed by chain[i],
    chain[i+1], .., chain[i+S-1] is a beta-gram whose every token after the first is a draft-model prediction (exact
    greedy text wherever the guesses before it were right).  One phrase per start i = 0 .. W-S+1, in that order."""
    W = len(src) - 1
    assert len(chain) == W + 1
    return [tuple(int(t) for t in [src[i]] + list(chain[i:i + S])) for i in range(0, W - S + 2)] if S >= 1 else []


class LookaheadDrafter:
    """Token-level drafting (Eq. 1) in which every draft forward also carries a window of W guessed tokens for
    the positions that follow, in the manner of the Jacobi iteration of lookahead decoding that Section 3.1 points to.

    The block of a draft forward is the text the draft model has not cached yet followed by the window, packed like
    one candidate suffix (Eq. 8 mask: window row i sees the text and window rows 1..i).  The real rows give the next
    draft token exactly as in plain drafting (the window rows are invisible to them); the window rows give the
    model's predictions under the guessed context.  Those predictions (a) become the next forward's guesses - the
    window slides with the text, one Jacobi step per forward; a window that holds the draft model's own greedy
    continuation is a fixed point - and (b) yield new phrases for the pool (window_phrases), inserted at once, so
    that the verification that follows can already look them up.  Drafts are exactly those of ModelDrafter."""

    def __init__(self, W, P, pool, width):
        self.W, self.P, self.pool, self.width = W, P, pool, width
        self.cache = tf.KVCache(W.desc)
        self.window = None
        self.calls = 0

    def draft(self, seq, gamma, step):
        c, S, out = self.cache, self.P.S, []
        if self.window is None:       # first guesses: the text's own last tokens (any tokens would do)
            tail = [int(t) for t in seq[-self.width:]] if self.width else []
            self.window = [int(seq[-1])] * (self.width - len(tail)) + tail
        feed = [int(t) for t in seq[c.length:]]
        for _ in range(gamma):
            n, L = len(feed), c.length
            cands = [list(self.window)] if self.width else []
            tokens, pos, group, visible = build_block(L, feed[0], feed[1:], cands)
            o = tf.argmax_rows(tf.forward(self.W, c, tokens, pos, visible))
            self.calls += 1
            c.length = L + n                                     # the window's K/V rows are left behind
            chain = [int(o[n - 1])] + [int(t) for t in o[n:n + self.width]]
            if self.width:
                for ph in window_phrases([feed[-1]] + self.window, chain, S):
                    self.pool.insert(ph)
                self.window = chain[1:]                          # predictions for the positions after the new token
            feed = [chain[0]]
            out.append(chain[0])
        return out

    def rollback(self, valid_len):
        self.cache.length = min(self.cache.length, valid_len)


class FixedDrafter:
    """Drafts supplied from outside (replay mode, hand traces): fn(seq, gamma, step) -> tokens."""

    def __init__(self, fn):
        self.fn = fn

    def draft(self, seq, gamma, step):
        return [int(t) for t in self.fn(seq, gamma, step)]

    def rollback(self, valid_len):
        pass


def generate(W, drafter, prompt, max_new, P, pool=None, trace=None):
    """Ouroboros greedy decoding, one iteration per loop turn: draft (Eq. 1), look up K phrases that
    start with d_gamma and pack them (Eq. 7), verify everything with one target forward (Eq. 2, Eq. 8),
    accept (Eq. 3, Eq. 9), compact the cache, harvest phrases (Section 3.3).  Passing a ``pool`` that
    already holds phrases reuses history (Section 3.4).  Returns (tokens, stats)."""
    gamma, S, beta = P.gamma, P.beta - 1, P.beta
    pool = PhrasePool(P.pool_sets, P.pool_ways, beta) if pool is None else pool
    pool.apply(prompt_ops(prompt, beta, P))
    cache = tf.KVCache(W.desc)
    prefill(W, cache, list(prompt[:-1]))
    seq, out = [int(t) for t in prompt], []
    stats = dict(target_calls=0, accepted=[], A=[], chosen=[], m=[], n_cand=[])
    step = 0
    while len(out) < max_new:
        L = cache.length                                   # seq[L] is the pending token
        d = drafter.draft(seq, gamma, step)
        cands = pool.lookup(d[-1], P.K)
        tokens, pos, group, visible = build_block(L, seq[L], d, cands)
        o = tf.argmax_rows(tf.forward(W, cache, tokens, pos, visible))
        A, j, m, accepted = accept(tokens, o, gamma, S, len(cands))
        moves = compact(cache, L, gamma, S, A, j, m)
        seq += accepted
        ops = harvest_ops(tokens, o, gamma, S, len(cands), A, seq, len(accepted), P)
        pool.apply(ops)
        drafter.rollback(L + min(A + 1, gamma))
        out += accepted
        stats["target_calls"] += 1
        for k, v in (("accepted", len(accepted)), ("A", A), ("chosen", j), ("m", m), ("n_cand", len(cands))):
            stats[k].append(v)
        if trace is not None:
            trace.append(dict(L=L, tokens=tokens, pos=pos, group=group, o=[int(t) for t in o], A=A, chosen=j, m=m,
                              accepted=list(accepted), moves=moves, ops=ops, pool=pool.export()))
        step += 1
        if P.eos_token >= 0 and P.eos_token in accepted:
            out = out[: len(out) - len(accepted) + accepted.index(P.eos_token) + 1]
            break
    out = out[:max_new]
    stats["eta"] = len(out) / max(1, stats["target_calls"])     # block efficiency (Appendix C)
    return out, stats
