"""The entry point that allocates nothing (ouro_lm_head_static).

Collected last on purpose: if it fails, a run that stops at the first failure has already run everything else.
Who needs it: users of this library who cannot hand it a workspace or let it allocate - a serving process whose
own arena owns all device memory, or a loop that must not risk the synchronisation an allocation can cause.  The
call keeps the GEMM's split-K scratch in a fixed 5 MiB array inside the library instead.

Expected values, first: logits = x . lm_head^T evaluated in float64 by numpy on the very bf16 inputs the call
gets (the definition of the LM-head pass, nothing of the CUDA path in it).  Second, as a cross-check between the
two entry points: a one-layer model whose output projections are zero leaves the residual stream equal to the
token embeddings, so the regular ouro_verify_forward computes logits = normalise(embedding rows) x lm_head^T; the
static call gets the same normalised rows and the same head and must agree to bf16 rounding.

Shapes are chosen so that the static array's split-K slots and counters are really used: with 32 CTAs a
vocabulary of 4000 (32 tiles) takes only whole tiles, 2048 (16 tiles) splits every tile between two CTAs, 4104
(33 tiles) leaves one ragged tile of 8 entries cut four ways, and a 64-wide model leaves fewer work items than
CTAs.  Every shape is run twice in a row with different rows, so a counter or a slot left over from the
previous call would show.
"""
import numpy as np
import pytest
import torch

from paper_2402_13720_b200 import binding, build, synth

pytestmark = pytest.mark.gpu
BF16_REL = 3e-2     # same bound as the parity tests: per row, relative to the largest |logit|


def _verify_forward_logits(desc, w, tokens):
    P = synth.DecodeParams(2, 3, 1, 4, 4, seed_prompt=False)
    eng = binding.Engine(desc, w, P)
    eng.assemble_causal(binding.OURO_TARGET, tokens)
    am, lg = eng.verify_forward(want_logits=True)
    torch.cuda.synchronize()
    out = am[: len(tokens)].clone(), lg[: len(tokens)].clone()
    eng.close()
    return out


def _check_against_definition(x, head, arg, logits):
    want = x.double().cpu().numpy() @ head.double().cpu().numpy().T            # float64, the definition
    got = logits.double().cpu().numpy()
    err = np.abs(got - want).max(axis=1)
    scale = np.abs(want).max(axis=1)
    assert (err <= BF16_REL * scale).all(), float((err / scale).max())
    srt = np.sort(want, axis=1)
    safe = (srt[:, -1] - srt[:, -2]) > 2 * err + 1e-9
    assert safe.sum() >= 1 and np.array_equal(arg.cpu().numpy()[safe], want.argmax(axis=1)[safe])
    assert torch.equal(arg.long(), logits.argmax(dim=1))                       # consistent with its own logits
    return err


@pytest.mark.parametrize("d_model,vocab", [(256, 4000), (256, 2048), (256, 4104), (64, 2048), (512, 1032)])
def test_static_scratch_head_equals_the_definition_twice(d_model, vocab):
    build.build()
    head = synth.tensor(21, 3, (vocab, d_model), 0.02, torch.bfloat16, "cuda:0")
    for call, rows in enumerate((37, 5, 128)):                                 # calls in a row, different sizes
        x = synth.tensor(22 + call, 4, (rows, d_model), 1.0, torch.bfloat16, "cuda:0")
        arg, logits = binding.lm_head_static(x, head, want_logits=True)
        _check_against_definition(x, head, arg, logits)
        arg2, _ = binding.lm_head_static(x, head)                              # without logits: same greedy tokens
        assert torch.equal(arg2, arg)


def test_static_scratch_head_matches_verify_forward_twice():
    build.build()
    desc = synth.ModelDesc(1, 256, 4, 4, 64, 256, 4104, 192, "bf16")
    w = synth.model_weights(desc, 11, device="cuda:0")
    w["layers"][0]["wo"].zero_()
    w["layers"][0]["w_down"].zero_()
    rng = np.random.default_rng(0)
    for call, rows in enumerate((37, 5)):                       # two calls in a row, different sizes
        tokens = rng.integers(0, desc.vocab, rows).astype(np.int32)
        ref_arg, ref_logits = _verify_forward_logits(desc, w, tokens)
        x = w["embed"][torch.as_tensor(tokens.astype(np.int64), device="cuda:0")].float()
        inv = 1.0 / torch.sqrt((x * x).mean(dim=1, keepdim=True) + desc.rms_eps)
        xn = (w["final_norm"].float() * (x * inv)).to(torch.bfloat16).contiguous()
        arg, logits = binding.lm_head_static(xn, w["lm_head"], want_logits=True)
        _check_against_definition(xn, w["lm_head"], arg, logits)
        err = (logits - ref_logits).abs().amax(dim=1)
        scale = ref_logits.abs().amax(dim=1)
        assert bool((err <= BF16_REL * scale).all()), (call, float((err / scale).max()))
        top2 = ref_logits.topk(2, dim=1).values
        safe = (top2[:, 0] - top2[:, 1]) > 2 * err + 1e-6
        assert int(safe.sum()) >= 1 and torch.equal(arg[safe], ref_arg[safe])


def test_static_scratch_head_breaks_exact_ties_towards_the_smallest_id():
    """Identical rows of the head give bit-identical logits; the greedy choice must then be the smallest id,
    whether the copies share a 128-entry tile or not."""
    build.build()
    d_model, vocab = 256, 2048
    head = synth.tensor(31, 3, (vocab, d_model), 0.02, torch.bfloat16, "cuda:0")
    x = synth.tensor(32, 4, (37, d_model), 1.0, torch.bfloat16, "cuda:0")
    win = (x[0].float() * 0.05).to(torch.bfloat16)               # a row whose logit for x[0] dominates
    for ids in ((700, 731, 1500), (1990, 130, 131)):
        h = head.clone()
        for i in ids:
            h[i] = win
        arg, logits = binding.lm_head_static(x, h, want_logits=True)
        assert len({float(logits[0, i]) for i in ids}) == 1 and int(logits[0].argmax()) in ids
        assert int(arg[0]) == min(ids)


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
