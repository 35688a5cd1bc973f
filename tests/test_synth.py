"""The seeded input generators: reproducible, device independent, with the stated statistics."""
import numpy as np
import torch

from paper_2402_13720_b200 import synth


def test_tensor_matches_python_integer_hash():
    t = synth.tensor(7, 33, (5, 9), 0.02, torch.float32)
    flat = t.flatten()
    for e in (0, 1, 17, 44):
        h = synth.hash_u64(7, 33, e)
        s = sum((h >> (16 * k)) & 0xFFFF for k in range(4)) - 131070
        assert flat[e].item() == np.float32(s) * np.float32(0.02 / synth._IH_SIGMA)


def test_tensor_statistics_and_chunking():
    a = synth.tensor(1, 2, (1 << 16,), 0.02)
    b = synth.tensor(1, 2, (1 << 16,), 0.02, chunk=1000)
    assert torch.equal(a, b)
    assert abs(a.mean().item()) < 5e-4 and abs(a.std().item() - 0.02) < 5e-4
    g = synth.tensor(1, 3, (4096,), 0.1, offset=1.0)
    assert abs(g.mean().item() - 1.0) < 0.01
    assert synth.tensor(1, 2, (64,), 0.02, torch.bfloat16).dtype == torch.bfloat16
    assert not torch.equal(a[:64], synth.tensor(2, 2, (64,), 0.02))


def test_prompt_recipe():
    p = synth.prompt(0, 512, 32, 0.5, 8, 8)
    assert p.dtype == np.int32 and len(p) == 32 and p.min() >= 0 and p.max() < 512
    assert np.array_equal(p, synth.prompt(0, 512, 32, 0.5, 8, 8))
    big = synth.prompt(1, 32000, 4096, 0.3, 8, 32)
    # copied spans make 8-grams repeat; a span-free prompt of Zipf tokens has almost none
    def rep(x):
        grams = [tuple(x[i:i + 8]) for i in range(len(x) - 7)]
        return 1.0 - len(set(grams)) / len(grams)
    assert rep(big) > 0.1 and rep(synth.prompt(1, 32000, 4096, 0.0, 8, 32)) < 0.02
    # Zipf head: the most frequent token covers several percent of a span-free text
    plain = synth.prompt(2, 32000, 8192, 0.0, 8, 32)
    assert np.bincount(plain).max() / len(plain) > 0.05


def test_configs():
    t, d, P, _ = synth.config("C2")
    assert P.block_max == 37 and t.layer_weight_elems() * 2 == 404750336
    t, d, P, _ = synth.config("C4")
    assert P.block_max == 69
    t, d, P, _ = synth.config("C1")
    assert P.block_max == 17 and d.n_layers == 1
