"""The entry point that allocates nothing (ouro_lm_head_static), against the regular verify forward.

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else.
Who needs it: users of this library who cannot hand it a workspace or let it allocate - a serving process whose
own arena owns all device memory, or a loop that must not risk the synchronisation an allocation can cause.  The
call keeps the GEMM's split-K scratch in a fixed 5 MiB array inside the library instead.

Reference: a one-layer model whose output projections are zero leaves the residual stream equal to the token
embeddings, so the regular ouro_verify_forward computes logits = normalise(embedding rows) x lm_head^T.  The
static call gets the same normalised rows and the same head and must give the same logits to bf16 rounding
(the two launches split K differently) and the same greedy tokens wherever the top-2 margin is not a rounding tie.
Two calls in a row check that the shared array is re-initialised correctly between calls.
"""
import numpy as np
import pytest
import torch

from paper_2402_13720_b200 import binding, build, synth

pytestmark = pytest.mark.gpu
BF16_REL = 3e-2     # same bound as the parity tests: per row, relative to the largest |logit|


def _reference(desc, w, tokens):
    P = synth.DecodeParams(2, 3, 1, 4, 4, seed_prompt=False)
    eng = binding.Engine(desc, w, P)
    eng.assemble_causal(binding.OURO_TARGET, tokens)
    am, lg = eng.verify_forward(want_logits=True)
    torch.cuda.synchronize()
    out = am[: len(tokens)].clone(), lg[: len(tokens)].clone()
    eng.close()
    return out


def test_static_scratch_head_matches_verify_forward_twice():
    build.build()
    desc = synth.ModelDesc(1, 256, 4, 4, 64, 256, 4000, 192, "bf16")
    w = synth.model_weights(desc, 11, device="cuda:0")
    w["layers"][0]["wo"].zero_()
    w["layers"][0]["w_down"].zero_()
    rng = np.random.default_rng(0)
    for call, rows in enumerate((37, 5)):                       # two calls in a row, different sizes
        tokens = rng.integers(0, desc.vocab, rows).astype(np.int32)
        ref_arg, ref_logits = _reference(desc, w, tokens)
        x = w["embed"][torch.as_tensor(tokens.astype(np.int64), device="cuda:0")].float()
        inv = 1.0 / torch.sqrt((x * x).mean(dim=1, keepdim=True) + desc.rms_eps)
        xn = (w["final_norm"].float() * (x * inv)).to(torch.bfloat16).contiguous()
        arg, logits = binding.lm_head_static(xn, w["lm_head"], want_logits=True)
        err = (logits - ref_logits).abs().amax(dim=1)
        scale = ref_logits.abs().amax(dim=1)
        assert bool((err <= BF16_REL * scale).all()), (call, float((err / scale).max()))
        top2 = ref_logits.topk(2, dim=1).values
        safe = (top2[:, 0] - top2[:, 1]) > 2 * err + 1e-6
        assert int(safe.sum()) >= 1 and torch.equal(arg[safe], ref_arg[safe])
        assert torch.equal(arg.long(), logits.argmax(dim=1))     # consistent with its own logits
        arg2, _ = binding.lm_head_static(xn, w["lm_head"])        # without logits: same greedy tokens
        assert torch.equal(arg2, arg)


def test_static_scratch_rejects_sizes_beyond_its_limits():
    build.build()
    x = torch.zeros((4, 128), dtype=torch.bfloat16, device="cuda:0")
    big = torch.zeros((8, 128), dtype=torch.bfloat16, device="cuda:0")
    lib = binding.lib()
    am = torch.zeros(4, dtype=torch.int32, device="cuda:0")
    rc = lib.ouro_lm_head_static(x.data_ptr(), big.data_ptr(), 4, 128, 65536 + 8, am.data_ptr(), None, None)
    assert rc == binding.OURO_EINVAL and b"static scratch" in lib.ouro_last_error(None)
    assert lib.ouro_lm_head_static(x.data_ptr(), big.data_ptr(), 129, 128, 8, am.data_ptr(), None, None) == binding.OURO_EINVAL
    assert lib.ouro_lm_head_static(x.data_ptr(), big.data_ptr(), 4, 100, 8, am.data_ptr(), None, None) == binding.OURO_EINVAL
