"""The input generators: determinism, storage format, and the statistics the recipes promise."""
import numpy as np
import torch

import lantern_inputs as li


def test_bf16_rounding_matches_torch():
    x = np.random.default_rng(1).normal(0, 3, 10000).astype(np.float32)
    x[:4] = [0.0, -0.0, np.inf, 1.00390625]  # last one is a round-to-even tie
    bits = li.f32_to_bf16_bits(x)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(bits, want)
    back = li.bf16_bits_to_f32(bits)
    assert np.array_equal(back, torch.from_numpy(x).to(torch.bfloat16).float().numpy())


def test_deterministic_and_seed_sensitive():
    a = li.config_verify_inputs("batch_chain", step=3, B=2, V=256)
    b = li.config_verify_inputs("batch_chain", step=3, B=2, V=256)
    c = li.config_verify_inputs("batch_chain", step=4, B=2, V=256)
    assert np.array_equal(a.target_logits, b.target_logits) and np.array_equal(a.draft_tokens, b.draft_tokens)
    assert not np.array_equal(a.target_logits, c.target_logits)
    assert a.target_logits.dtype == np.uint16 and a.target_logits.shape == (2, 2, 8, 256)
    assert a.uniforms.min() >= 0.0 and a.uniforms.max() < 1.0


def test_tree_shape():
    par = li.tree_parents(5, 60, depth=6, seed=3)
    for b in range(5):
        depth = np.zeros(60, int)
        for i in range(60):
            assert -1 <= par[b, i] < i
            depth[i] = 1 if par[b, i] < 0 else depth[par[b, i]] + 1
        assert depth.max() == 6 and list(par[b, :6]) == [-1, 0, 1, 2, 3, 4]
    inp = li.config_verify_inputs("single_image", B=2, V=512)
    for b in range(2):
        for c in range(61):
            kids = np.nonzero(inp.tree_parents[b] == c - 1)[0]
            assert len(set(inp.draft_tokens[b, kids].tolist())) == kids.size  # siblings are distinct tokens


def test_codebooks():
    cb = li.codebook_gaussian(100, 8)
    np.testing.assert_allclose(np.linalg.norm(cb.astype(np.float64), axis=1), 1.0, atol=1e-6)
    cl = li.codebook_clustered(2048, 16)
    d_same = np.linalg.norm(cl[0] - cl[512])
    d_other = np.linalg.norm(cl[0] - cl[1])
    assert d_same < 1.0 < d_other


def test_tokens_follow_the_drafter():
    # Gumbel-max draws: the empirical law of the first draft token matches softmax(draft row 0)
    V, B = 16, 1
    hits = np.zeros(V)
    base = li.verify_inputs(B, 1, V, dtype=li.F32, has_uncond=False, sigma_target=1.0, sigma_draft=0.0, seed=5)
    z = base.draft_logits[0, 0].astype(np.float64)
    p = np.exp(z - z.max()); p /= p.sum()
    g = np.random.default_rng(0)
    n = 20000
    pert = z[None, :] + li._gumbel(g, (n, V))
    hits = np.bincount(pert.argmax(1), minlength=V)
    assert np.abs(hits / n - p).max() < 0.02
