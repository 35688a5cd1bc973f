"""Seeded synthetic inputs: model shapes, weights, KV caches, prompts, corrupted drafts.

Everything here is input generation only.  It holds none of the decoding method's
arithmetic (no attention, no acceptance, no pool logic), so both the CUDA path and the
CPU oracle may be fed from it.  All randomness is counter based: element ``e`` of tensor
``tid`` under ``seed`` is a pure function of ``(seed, tid, e)``, evaluated with integer
operations only (splitmix64 finaliser), so CPU and CUDA tensors are bit identical.

Stand-ins (the paper evaluates trained Yi / Llama-2 pairs on public datasets, Section 4.1;
neither weights nor datasets are available, so shapes and statistics are mimicked):
  * weights ~ N(0, 0.02) approximated by a 4-term Irwin-Hall sum (bounded at 3.46 sigma),
    norm gains 1 + 0.1 z so that a dropped gain changes the result;
  * prompts: Zipf(1.1) token ranks under a seeded rank->id permutation, with spans copied
    from earlier in the sequence (the phrase locality the method exploits, Appendix F).
"""
from __future__ import annotations

import dataclasses
import math

import numpy as np
import torch

_M64 = (1 << 64) - 1
_GOLD = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB
_IH_SIGMA = math.sqrt(4.0 * (65536.0 ** 2 - 1.0) / 12.0)  # std of the sum of four uniform u16


def _signed(u: int) -> int:
    u &= _M64
    return u - (1 << 64) if u >= (1 << 63) else u


def mix64(z: int) -> int:
    """splitmix64 output function on a Python integer (mod 2^64)."""
    z = (z + _GOLD) & _M64
    z = ((z ^ (z >> 30)) * _MUL1) & _M64
    z = ((z ^ (z >> 27)) * _MUL2) & _M64
    return z ^ (z >> 31)


def _lsr(z: torch.Tensor, k: int) -> torch.Tensor:
    return (z >> k) & ((1 << (64 - k)) - 1)


def _mix64_t(z: torch.Tensor) -> torch.Tensor:
    """splitmix64 output function on an int64 tensor (two's-complement wrap-around)."""
    z = z + _signed(_GOLD)
    z = (z ^ _lsr(z, 30)) * _signed(_MUL1)
    z = (z ^ _lsr(z, 27)) * _signed(_MUL2)
    return z ^ _lsr(z, 31)


def stream_base(seed: int, tid: int) -> int:
    return mix64((seed * _GOLD + tid * _MUL1 + 0x1234567) & _M64)


def hash_u64(seed: int, tid: int, e: int) -> int:
    """Python-int twin of the per-element hash used by :func:`tensor` (tests cross-check it)."""
    return mix64((stream_base(seed, tid) + e) & _M64)


def tensor(seed: int, tid: int, shape, scale: float, dtype=torch.float32, device="cpu",
           offset: float = 0.0, chunk: int = 1 << 24) -> torch.Tensor:
    """offset + scale * z with z approximately N(0,1); fp32 arithmetic, then one cast to ``dtype``."""
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=dtype, device=device)
    base = _signed(stream_base(seed, tid))
    c = np.float32(scale / _IH_SIGMA)
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        h = _mix64_t(torch.arange(lo, hi, dtype=torch.int64, device=device) + base)
        s = (h & 0xFFFF) + (_lsr(h, 16) & 0xFFFF) + (_lsr(h, 32) & 0xFFFF) + (_lsr(h, 48) & 0xFFFF) - 131070
        w = s.to(torch.float32) * float(c)
        if offset != 0.0:
            w = w + float(np.float32(offset))
        out[lo:hi] = w.to(dtype)
    return out.view(*shape)


@dataclasses.dataclass(frozen=True)
class ModelDesc:
    n_layers: int
    d_model: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    d_ffn: int
    vocab: int
    max_seq: int
    dtype: str = "f32"          # "f32" | "bf16"
    rope_theta: float = 10000.0
    rms_eps: float = 1e-5

    @property
    def torch_dtype(self):
        return torch.float32 if self.dtype == "f32" else torch.bfloat16

    @property
    def d_q(self):
        return self.n_heads * self.head_dim

    @property
    def d_kv(self):
        return self.n_kv_heads * self.head_dim

    def layer_weight_elems(self) -> int:
        d, F = self.d_model, self.d_ffn
        return d * self.d_q * 2 + 2 * d * self.d_kv + 3 * d * F

    def early_exit(self, n_layers: int) -> "ModelDesc":
        return dataclasses.replace(self, n_layers=n_layers)


@dataclasses.dataclass(frozen=True)
class DecodeParams:
    gamma: int                   # draft length
    beta: int                    # phrase length including its first token (= d_gamma)
    K: int                       # candidates per step
    pool_sets: int = 128
    pool_ways: int = 32
    harvest_matched: bool = True      # matched sub-segments of the discarded draft (Section 3.3)
    harvest_candidates: bool = True   # corrected candidates (Section 3.3, second paragraph)
    harvest_accepted: bool = True     # beta-grams of the accepted text (extension, off in paper-pure mode)
    seed_prompt: bool = True          # beta-grams of the prompt (extension, off in paper-pure mode)
    draft_phrases: bool = False       # the draft model drafts phrase by phrase (Section 3.1)
    window: int = 0                   # lookahead window riding along every draft forward (phrase generation, Section 3.1)
    eos_token: int = -1

    @property
    def S(self):
        return self.beta - 1

    @property
    def block_max(self):
        return 1 + self.gamma + self.K * self.S

    def paper_pure(self) -> "DecodeParams":
        return dataclasses.replace(self, harvest_accepted=False, seed_prompt=False)


LAYER_TENSORS = ("attn_norm", "wq", "wk", "wv", "wo", "ffn_norm", "w_gate", "w_up", "w_down")


def layer_shapes(m: ModelDesc) -> dict:
    d, F = m.d_model, m.d_ffn
    return {"attn_norm": (d,), "wq": (m.d_q, d), "wk": (m.d_kv, d), "wv": (m.d_kv, d), "wo": (d, m.d_q),
            "ffn_norm": (d,), "w_gate": (F, d), "w_up": (F, d), "w_down": (d, F)}


def model_weights(m: ModelDesc, seed: int, device="cpu", layers=None, with_head: bool = True) -> dict:
    """{'embed','final_norm','lm_head', 'layers': [ {name: tensor} ]}; row-major [out, in] matrices."""
    dt = m.torch_dtype
    w = {}
    if with_head:
        w["embed"] = tensor(seed, 1, (m.vocab, m.d_model), 0.02, dt, device)
        w["final_norm"] = tensor(seed, 2, (m.d_model,), 0.1, dt, device, offset=1.0)
        w["lm_head"] = tensor(seed, 3, (m.vocab, m.d_model), 0.02, dt, device)
    w["layers"] = []
    for l in (range(m.n_layers) if layers is None else layers):
        lw = {}
        for k, (name, shp) in enumerate(layer_shapes(m).items()):
            tid = 16 * (l + 1) + k
            if name.endswith("norm"):
                lw[name] = tensor(seed, tid, shp, 0.1, dt, device, offset=1.0)
            else:
                lw[name] = tensor(seed, tid, shp, 0.02, dt, device)
        w["layers"].append(lw)
    return w


def kv_fill(m: ModelDesc, seed: int, length: int, device="cpu"):
    """Random K and V caches [n_layers, max_seq, n_kv_heads, head_dim]; slots >= length are zero.
    Unit-variance entries, treated as already-rotated keys (verify microbenchmark input)."""
    dt = m.torch_dtype
    shp = (m.n_layers, m.max_seq, m.n_kv_heads, m.head_dim)
    k = torch.zeros(shp, dtype=dt, device=device)
    v = torch.zeros(shp, dtype=dt, device=device)
    for l in range(m.n_layers):
        k[l, :length] = tensor(seed, 1000 + 2 * l, (length, m.n_kv_heads, m.head_dim), 1.0, dt, device)
        v[l, :length] = tensor(seed, 1001 + 2 * l, (length, m.n_kv_heads, m.head_dim), 1.0, dt, device)
    return k, v


def _uniform(seed: int, tid: int, e: int) -> float:
    return (hash_u64(seed, tid, e) >> 11) / float(1 << 53)


def prompt(seed: int, vocab: int, n: int, copy_frac: float, span_lo: int, span_hi: int,
           zipf_s: float = 1.1) -> np.ndarray:
    """Zipf(zipf_s) tokens with LZ-style copied spans covering about ``copy_frac`` of the text."""
    ranks = np.arange(1, vocab + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-zipf_s))
    cdf /= cdf[-1]
    keys = np.array([hash_u64(seed, 50, r) for r in range(vocab)], dtype=np.uint64)
    perm = np.argsort(keys, kind="stable").astype(np.int32)       # rank -> token id
    mean_len = 0.5 * (span_lo + span_hi)
    p_copy = copy_frac / (copy_frac + mean_len * (1.0 - copy_frac)) if copy_frac > 0 else 0.0
    out: list[int] = []
    e = 0
    while len(out) < n:
        u = _uniform(seed, 51, e)
        h = hash_u64(seed, 52, e)
        e += 1
        if len(out) >= span_lo and u < p_copy:
            length = span_lo + (h & 0xFFFF) % (span_hi - span_lo + 1)
            src = (h >> 16) % len(out)
            for k in range(length):
                if len(out) >= n:
                    break
                out.append(out[src + k])      # may run into the tokens just copied (overlapping copy)
        else:
            r = int(np.searchsorted(cdf, _uniform(seed, 53, e), side="left"))
            out.append(int(perm[min(r, vocab - 1)]))
    return np.asarray(out[:n], dtype=np.int32)


def corrupt_drafts(seed: int, truth: np.ndarray, start: int, gamma: int, vocab: int,
                   p_sub: float, p_skip: float, step: int) -> np.ndarray:
    """Replay drafter: gamma draft tokens read from a recorded continuation ``truth`` starting at
    ``start``, with seeded substitutions (prob p_sub per token) and single-token skips (prob
    p_skip per token, shifting the rest: the misplacement pattern of Section 3.3).  Stand-in for a
    trained draft model; positions past the end of ``truth`` are filled with hashed tokens."""
    out = np.empty(gamma, dtype=np.int32)
    src = start
    for i in range(gamma):
        e = step * 64 + i
        if _uniform(seed, 60, e) < p_skip:
            src += 1
        if src < len(truth) and _uniform(seed, 61, e) >= p_sub:
            out[i] = truth[src]
        else:
            out[i] = hash_u64(seed, 62, e) % vocab
        src += 1
    return out


# ---- the five workload configurations (shapes only) ---------------------------------------------

def config(name: str):
    """Returns (target ModelDesc, draft ModelDesc or None, DecodeParams, prompt recipe dict)."""
    if name == "C1":   # tiny fp32 pair; draft = target's embedding + first layer (early exit)
        t = ModelDesc(2, 128, 4, 4, 32, 344, 512, 256, "f32")
        return t, t.early_exit(1), DecodeParams(4, 4, 4, 128, 32), dict(n=32, copy_frac=0.5, span=(8, 8), gen=64)
    if name == "C2":   # one 7B-shaped layer, verify microbenchmark; vocab as in the 7B configuration
        t = ModelDesc(1, 4096, 32, 32, 128, 11008, 32000, 4096 + 64, "bf16")
        return t, None, DecodeParams(4, 9, 4, 128, 32), dict(n=0, copy_frac=0.0, span=(8, 8), gen=0)
    if name == "C3":
        t = ModelDesc(32, 4096, 32, 32, 128, 11008, 32000, 640, "bf16")
        s = ModelDesc(22, 2048, 32, 4, 64, 5632, 32000, 640, "bf16")
        return t, s, DecodeParams(4, 9, 4, 128, 32), dict(n=256, copy_frac=0.3, span=(8, 32), gen=256)
    if name == "C4":
        t = ModelDesc(60, 7168, 56, 8, 128, 20480, 64000, 1152, "bf16")
        s = ModelDesc(32, 4096, 32, 4, 128, 11008, 64000, 1152, "bf16")
        return t, s, DecodeParams(4, 9, 8, 128, 32), dict(n=512, copy_frac=0.3, span=(8, 32), gen=512)
    if name == "C5":
        t = ModelDesc(80, 8192, 64, 8, 128, 28672, 32000, 1152, "bf16")
        s = ModelDesc(32, 4096, 32, 32, 128, 11008, 32000, 1152, "bf16")
        return t, s, DecodeParams(4, 9, 4, 128, 32), dict(n=512, copy_frac=0.3, span=(8, 32), gen=512)
    raise KeyError(name)
