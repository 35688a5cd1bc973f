"""ctypes binding of libouro.so: argument marshalling only, every step runs in the CUDA library.

``lib()`` exposes the functions of include/ouro.h under their own names, with ctypes signatures, taking raw
pointers (ints) or ctypes objects.  ``Engine`` is a convenience holder that lets PyTorch allocate the
device memory (weights stay the caller's tensors; KV caches and workspace are torch tensors owned by the
Engine) and passes ``tensor.data_ptr()`` values down.  There is no fallback: without the built library,
or without a CUDA device for anything that computes, calls raise.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

from . import synth

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libouro.so")
_lib = None

OURO_OK, OURO_EINVAL, OURO_ENOMEM, OURO_ECAPACITY, OURO_ECUDA, OURO_ETIMEOUT, OURO_ESTATE = range(7)
OURO_F32, OURO_BF16 = 0, 1
OURO_TARGET, OURO_DRAFT = 0, 1
OURO_MAX_ROWS, OURO_MAX_BETA, OURO_MAX_K, OURO_MAX_GAMMA = 128, 16, 16, 32
OURO_HARVEST_MATCHED, OURO_HARVEST_CANDIDATES, OURO_HARVEST_ACCEPTED, OURO_SEED_PROMPT, OURO_DRAFT_PHRASES = 1, 2, 4, 8, 16


class ModelDescC(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "d_model", "n_heads", "n_kv_heads", "head_dim", "d_ffn",
                                           "vocab", "max_seq", "dtype")] + [("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class ModelMemC(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, C.POINTER(C.c_void_p)) for n in synth.LAYER_TENSORS] + \
               [("k_cache", C.c_void_p), ("v_cache", C.c_void_p)]


class ParamsC(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("gamma", "beta", "K", "pool_sets", "pool_ways")] + \
               [("flags", C.c_uint32), ("eos_token", C.c_int32), ("window", C.c_int32)]


class StatsC(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_tokens", "target_calls", "draft_calls", "full_accepts", "suffix_tokens",
                                           "candidates")] + [(n, C.c_float) for n in ("ms_total", "ms_target", "ms_draft")]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


DRAFTER_FN = C.CFUNCTYPE(C.c_int, C.c_void_p, C.POINTER(C.c_int32), C.c_int32, C.c_int32, C.c_int32, C.POINTER(C.c_int32))

_I32P, _U64P, _F32P = C.POINTER(C.c_int32), C.POINTER(C.c_uint64), C.POINTER(C.c_float)
_SIGNATURES = {
    "ouro_strerror": (C.c_char_p, [C.c_int]),
    "ouro_last_error": (C.c_char_p, [C.c_void_p]),
    "ouro_workspace_bytes": (C.c_size_t, [C.POINTER(ModelDescC), C.POINTER(ModelDescC), C.POINTER(ParamsC)]),
    "ouro_create": (C.c_int, [C.POINTER(ModelDescC), C.POINTER(ModelMemC), C.POINTER(ModelDescC), C.POINTER(ModelMemC),
                              C.POINTER(ParamsC), C.c_void_p, C.c_size_t, C.c_void_p, C.POINTER(C.c_void_p)]),
    "ouro_destroy": (C.c_int, [C.c_void_p]),
    "ouro_reset": (C.c_int, [C.c_void_p, C.c_int]),
    "ouro_prefill": (C.c_int, [C.c_void_p, _I32P, C.c_int32]),
    "ouro_set_state": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32]),
    "ouro_get_state": (C.c_int, [C.c_void_p, _I32P, _I32P, _I32P]),
    "ouro_set_drafter": (C.c_int, [C.c_void_p, DRAFTER_FN, C.c_void_p]),
    "ouro_phrase_lookup": (C.c_int, [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]),
    "ouro_phrase_update": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32]),
    "ouro_pool_export": (C.c_int, [C.c_void_p, _I32P, _U64P, _I32P]),
    "ouro_pool_import": (C.c_int, [C.c_void_p, _I32P, C.c_int32]),
    "ouro_assemble_candidates": (C.c_int, [C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ouro_assemble_causal": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_int32]),
    "ouro_block_get": (C.c_int, [C.c_void_p, C.c_int, _I32P, _I32P, _I32P, _U64P, _I32P]),
    "ouro_verify_forward": (C.c_int, [C.c_void_p, C.c_int, C.c_void_p, C.c_void_p]),
    "ouro_accept_and_compact": (C.c_int, [C.c_void_p, C.c_void_p, _I32P, _I32P, _I32P, _I32P]),
    "ouro_verify_step": (C.c_int, [C.c_void_p, C.c_void_p, _I32P, _I32P, _I32P, _I32P]),
    "ouro_advance": (C.c_int, [C.c_void_p, C.c_int, C.c_int32]),
    "ouro_draft": (C.c_int, [C.c_void_p, C.c_void_p]),
    "ouro_kernel_launches": (C.c_uint64, []),
    "ouro_lm_head_static": (C.c_int, [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]),
    "ouro_profile_enable": (C.c_int, [C.c_void_p, C.c_int]),
    "ouro_debug_set_wait_limit": (C.c_int, [C.c_void_p, C.c_int64]),
    "ouro_profile_read": (C.c_int, [C.c_void_p, _F32P, _I32P]),
    "ouro_generate": (C.c_int, [C.c_void_p, _I32P, C.c_int32, C.c_int32, C.c_int32, _I32P, _I32P, C.POINTER(StatsC)]),
    "ouro_generate_vanilla": (C.c_int, [C.c_void_p, _I32P, C.c_int32, C.c_int32, _I32P, _I32P, C.POINTER(StatsC)]),
}


def lib():
    """The loaded shared library; raises if it has not been built (there is no other implementation)."""
    global _lib
    if _lib is None:
        path = os.environ.get("OURO_LIB") or _LIB_PATH     # OURO_LIB: another build of the same library (trace.py)
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2402_13720_b200.build`")
        L = C.CDLL(path)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype, fn.argtypes = res, args
        _lib = L
    return _lib


def exported_names():
    return sorted(_SIGNATURES)


class OuroError(RuntimeError):
    def __init__(self, status, ctx=None):
        self.status = status
        text = lib().ouro_strerror(status).decode()
        detail = lib().ouro_last_error(ctx).decode()
        super().__init__(f"ouro status {status} ({text}): {detail}")


def _check(status, ctx=None):
    if status != OURO_OK:
        raise OuroError(status, ctx)


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(_I32P)


def desc_c(m: synth.ModelDesc) -> ModelDescC:
    return ModelDescC(m.n_layers, m.d_model, m.n_heads, m.n_kv_heads, m.head_dim, m.d_ffn, m.vocab, m.max_seq,
                      OURO_F32 if m.dtype == "f32" else OURO_BF16, m.rope_theta, m.rms_eps)


def params_c(p: synth.DecodeParams) -> ParamsC:
    flags = (OURO_HARVEST_MATCHED if p.harvest_matched else 0) | (OURO_HARVEST_CANDIDATES if p.harvest_candidates else 0) | \
            (OURO_HARVEST_ACCEPTED if p.harvest_accepted else 0) | (OURO_SEED_PROMPT if p.seed_prompt else 0) | \
            (OURO_DRAFT_PHRASES if getattr(p, "draft_phrases", False) else 0)
    return ParamsC(p.gamma, p.beta, p.K, p.pool_sets, p.pool_ways, flags, p.eos_token, getattr(p, "window", 0))


def lm_head_static(x: torch.Tensor, lm_head: torch.Tensor, want_logits: bool = False):
    """LM-head pass for callers that cannot allocate: the library's own 5 MiB static array serves as scratch
    (see ouro_lm_head_static in include/ouro.h).  x [rows, d] and lm_head [vocab, d] are bf16 CUDA tensors; the
    outputs are allocated here by torch only because this is the Python convenience wrapper - the C call itself
    allocates nothing.  Returns (argmax int32 [rows], logits fp32 [rows, vocab] or None)."""
    assert x.is_cuda and lm_head.is_cuda and x.dtype == torch.bfloat16 and lm_head.dtype == torch.bfloat16
    assert x.is_contiguous() and lm_head.is_contiguous() and x.shape[1] == lm_head.shape[1]
    rows, d = x.shape
    vocab = lm_head.shape[0]
    argmax = torch.empty(rows, dtype=torch.int32, device=x.device)
    logits = torch.empty((rows, vocab), dtype=torch.float32, device=x.device) if want_logits else None
    with torch.cuda.device(x.device):
        _check(lib().ouro_lm_head_static(x.data_ptr(), lm_head.data_ptr(), rows, d, vocab, argmax.data_ptr(),
                                         logits.data_ptr() if want_logits else None,
                                         torch.cuda.current_stream(x.device).cuda_stream))
    return argmax, logits


class _ModelMem:
    """Keeps the ctypes pointer arrays (and the tensors behind them) alive."""

    def __init__(self, m: synth.ModelDesc, w: dict, device):
        self.w = w
        self.k_cache = torch.zeros((m.n_layers, m.max_seq, m.n_kv_heads, m.head_dim), dtype=m.torch_dtype, device=device)
        self.v_cache = torch.zeros_like(self.k_cache)
        self.arrays = {}
        for name in synth.LAYER_TENSORS:
            ptrs = [w["layers"][l][name].data_ptr() for l in range(m.n_layers)]
            self.arrays[name] = (C.c_void_p * m.n_layers)(*ptrs)
        for t in [w["embed"], w["final_norm"], w["lm_head"]] + [lw[n] for lw in w["layers"][: m.n_layers] for n in synth.LAYER_TENSORS]:
            assert t.is_cuda and t.is_contiguous() and t.dtype == m.torch_dtype and t.data_ptr() % 16 == 0
        self.c = ModelMemC(w["embed"].data_ptr(), w["final_norm"].data_ptr(), w["lm_head"].data_ptr(),
                           *[C.cast(self.arrays[n], C.POINTER(C.c_void_p)) for n in synth.LAYER_TENSORS],
                           self.k_cache.data_ptr(), self.v_cache.data_ptr())


class Engine:
    """One decoding stream on one GPU.  Method names follow include/ouro.h without the ``ouro_`` prefix."""

    def __init__(self, target: synth.ModelDesc, target_w: dict, params: synth.DecodeParams,
                 draft: synth.ModelDesc | None = None, draft_w: dict | None = None, device="cuda:0"):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this library has no CPU path")
        self.L = lib()
        self.device = torch.device(device)
        self.target_desc, self.draft_desc, self.params = target, draft, params
        self.tm = _ModelMem(target, target_w, self.device)
        self.dm = _ModelMem(draft, draft_w, self.device) if draft is not None else None
        self._td, self._pd = desc_c(target), params_c(params)
        self._dd = desc_c(draft) if draft is not None else None
        nbytes = self.L.ouro_workspace_bytes(C.byref(self._td), C.byref(self._dd) if self._dd else None, C.byref(self._pd))
        if nbytes == 0:
            raise OuroError(OURO_EINVAL)
        self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
        ws = (self.workspace.data_ptr() + 255) & ~255
        self.stream = torch.cuda.current_stream(self.device)
        ctx = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.L.ouro_create(C.byref(self._td), C.byref(self.tm.c), C.byref(self._dd) if self._dd else None,
                                      C.byref(self.dm.c) if self.dm else None, C.byref(self._pd), ws, nbytes,
                                      self.stream.cuda_stream, C.byref(ctx)))
        self.ctx = ctx
        self._drafter_cb = None
        R = OURO_MAX_ROWS
        self.argmax = torch.zeros(R, dtype=torch.int32, device=self.device)
        self.logits = torch.zeros((R, target.vocab), dtype=torch.float32, device=self.device)
        self.draft_tokens = torch.zeros(max(1, params.gamma), dtype=torch.int32, device=self.device)
        self.suffix = torch.zeros(max(1, params.K * params.S), dtype=torch.int32, device=self.device)
        self.count = torch.zeros(1, dtype=torch.int32, device=self.device)

    def close(self):
        if getattr(self, "ctx", None):
            self.L.ouro_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _ck(self, status):
        _check(status, self.ctx)

    # ---- state -------------------------------------------------------------------------------
    def reset(self, keep_pool=False):
        self._ck(self.L.ouro_reset(self.ctx, int(keep_pool)))

    def prefill(self, prompt):
        a, p = _i32(prompt)
        self._ck(self.L.ouro_prefill(self.ctx, p, len(a)))

    def set_state(self, cache_len, pending):
        self._ck(self.L.ouro_set_state(self.ctx, cache_len, pending))

    def get_state(self):
        t, d, p = C.c_int32(), C.c_int32(), C.c_int32()
        self._ck(self.L.ouro_get_state(self.ctx, C.byref(t), C.byref(d), C.byref(p)))
        return t.value, d.value, p.value

    def set_drafter(self, fn):
        """fn(seq: np.ndarray, gamma: int, step: int) -> gamma tokens, or None to remove."""
        if fn is None:
            self._drafter_cb = None
            self._ck(self.L.ouro_set_drafter(self.ctx, C.cast(None, DRAFTER_FN), None))
            return

        def cb(user, seq, n, gamma, step, out):
            try:
                toks = fn(np.ctypeslib.as_array(seq, shape=(n,)), gamma, step)
                for i in range(gamma):
                    out[i] = int(toks[i])
                return 0
            except Exception:
                return 1

        self._drafter_cb = DRAFTER_FN(cb)
        self._ck(self.L.ouro_set_drafter(self.ctx, self._drafter_cb, None))

    # ---- pool --------------------------------------------------------------------------------
    def phrase_lookup(self, key, K=None):
        K = self.params.K if K is None else K
        self._ck(self.L.ouro_phrase_lookup(self.ctx, int(key), K, self.suffix.data_ptr(), self.count.data_ptr()))
        n = int(self.count.item())
        return self.suffix[: n * self.params.S].view(n, self.params.S).cpu().numpy()

    def phrase_update(self, ngrams):
        t = torch.as_tensor(np.ascontiguousarray(ngrams, dtype=np.int32).reshape(-1, self.params.beta), device=self.device)
        self._ck(self.L.ouro_phrase_update(self.ctx, t.data_ptr(), t.shape[0]))
        torch.cuda.current_stream(self.device).synchronize()

    def pool_export(self):
        cap = self.params.pool_sets * self.params.pool_ways
        ng = np.zeros((cap, self.params.beta), dtype=np.int32)
        st = np.zeros(cap, dtype=np.uint64)
        n = C.c_int32()
        self._ck(self.L.ouro_pool_export(self.ctx, ng.ctypes.data_as(_I32P), st.ctypes.data_as(_U64P), C.byref(n)))
        return ng[: n.value], st[: n.value]

    def pool_import(self, ngrams):
        a, p = _i32(np.asarray(ngrams).reshape(-1, self.params.beta))
        self._ck(self.L.ouro_pool_import(self.ctx, p, a.shape[0]))

    # ---- one step ----------------------------------------------------------------------------
    def draft(self):
        self._ck(self.L.ouro_draft(self.ctx, self.draft_tokens.data_ptr()))
        return self.draft_tokens

    def assemble_candidates(self, draft=None, lookup_here=True):
        """draft: gamma tokens (host) or None to use the tokens left by draft().  lookup_here=False packs the
        candidates left in self.suffix/self.count by phrase_lookup()."""
        if draft is not None:
            self.draft_tokens[: self.params.gamma] = torch.as_tensor(np.asarray(draft, dtype=np.int32), device=self.device)
        suf, cnt = (None, None) if lookup_here else (self.suffix.data_ptr(), self.count.data_ptr())
        self._ck(self.L.ouro_assemble_candidates(self.ctx, self.draft_tokens.data_ptr(), suf, cnt))

    def assemble_causal(self, which, tokens):
        t = torch.as_tensor(np.asarray(tokens, dtype=np.int32), device=self.device)
        self._keep = t
        self._ck(self.L.ouro_assemble_causal(self.ctx, which, t.data_ptr(), t.numel()))

    def block_get(self, which=OURO_TARGET):
        R = OURO_MAX_ROWS
        tok, pos, grp = (np.zeros(R, dtype=np.int32) for _ in range(3))
        mask = np.zeros((R, 2), dtype=np.uint64)
        B = C.c_int32()
        self._ck(self.L.ouro_block_get(self.ctx, which, tok.ctypes.data_as(_I32P), pos.ctypes.data_as(_I32P),
                                       grp.ctypes.data_as(_I32P), mask.ctypes.data_as(_U64P), C.byref(B)))
        b = B.value
        return tok[:b], pos[:b], grp[:b], mask[:b]

    def verify_forward(self, which=OURO_TARGET, want_logits=False):
        self._ck(self.L.ouro_verify_forward(self.ctx, which, self.argmax.data_ptr(),
                                            self.logits.data_ptr() if want_logits else None))
        return self.argmax, (self.logits if want_logits else None)

    def accept_and_compact(self, argmax=None):
        o = self.argmax if argmax is None else argmax
        n, ch, A = C.c_int32(), C.c_int32(), C.c_int32()
        acc = np.zeros(OURO_MAX_GAMMA + OURO_MAX_BETA, dtype=np.int32)
        self._ck(self.L.ouro_accept_and_compact(self.ctx, o.data_ptr(), C.byref(n), C.byref(ch), C.byref(A),
                                                acc.ctypes.data_as(_I32P)))
        return n.value, ch.value, A.value, acc[: n.value].copy()

    def verify_step(self):
        """assemble_candidates + verify_forward + accept_and_compact in one library call, on the tokens in
        self.draft_tokens.  Returns (n_accepted, chosen, accurate, accepted tokens as a view that the next call reuses)."""
        if not hasattr(self, "_vs"):
            self._vs = (C.c_int32(), C.c_int32(), C.c_int32(), np.zeros(OURO_MAX_GAMMA + OURO_MAX_BETA, dtype=np.int32))
            self._vs_args = (self.draft_tokens.data_ptr(), C.byref(self._vs[0]), C.byref(self._vs[1]), C.byref(self._vs[2]),
                             self._vs[3].ctypes.data_as(_I32P))
        rc = self.L.ouro_verify_step(self.ctx, *self._vs_args)
        if rc != OURO_OK:
            raise OuroError(rc, self.ctx)
        n = self._vs[0].value
        return n, self._vs[1].value, self._vs[2].value, self._vs[3][:n]

    def advance(self, which, n):
        self._ck(self.L.ouro_advance(self.ctx, which, n))

    # ---- measurement -------------------------------------------------------------------------
    PROF = dict(off=-1, embed=0, norm=1, qkv=2, rope=3, attention=4, wo=5, gateup=6, down=7, head=8, argmax=9, forward=10, gemm=11)

    def profile_enable(self, kernel_class):
        self._ck(self.L.ouro_profile_enable(self.ctx, self.PROF[kernel_class] if isinstance(kernel_class, str) else kernel_class))

    def profile_read(self):
        ms, n = C.c_float(), C.c_int32()
        self._ck(self.L.ouro_profile_read(self.ctx, C.byref(ms), C.byref(n)))
        return ms.value, n.value

    def set_wait_limit(self, polls):
        self._ck(self.L.ouro_debug_set_wait_limit(self.ctx, int(polls)))

    # ---- loops -------------------------------------------------------------------------------
    def generate(self, prompt, max_new, keep_pool=False):
        a, p = _i32(prompt)
        out = np.zeros(max(1, max_new), dtype=np.int32)
        n, st = C.c_int32(), StatsC()
        self._ck(self.L.ouro_generate(self.ctx, p, len(a), max_new, int(keep_pool), out.ctypes.data_as(_I32P),
                                      C.byref(n), C.byref(st)))
        return out[: n.value].copy(), st.as_dict()

    def generate_vanilla(self, prompt, max_new):
        a, p = _i32(prompt)
        out = np.zeros(max(1, max_new), dtype=np.int32)
        n, st = C.c_int32(), StatsC()
        self._ck(self.L.ouro_generate_vanilla(self.ctx, p, len(a), max_new, out.ctypes.data_as(_I32P), C.byref(n), C.byref(st)))
        return out[: n.value].copy(), st.as_dict()
