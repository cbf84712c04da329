"""The shared input generator: bulk C fill against the scalar recipe, and the small seeded draws."""
import numpy as np
import torch

import synth


def test_bulk_fill_matches_scalar_recipe():
    Z = synth.normal_table()
    assert Z.shape == (65536,) and Z[0] < -4.0 and abs(Z[32768]) < 1e-4 and np.all(np.diff(Z) > 0)
    seed, tid = 0x1234567890, 77
    t32 = synth.fill((5, 13), seed, tid, 0.02, "f32", 0.01).flatten()
    t16 = synth.fill((5, 13), seed, tid, 0.02, "bf16", 0.01).flatten()
    for i in range(65):
        g, lane = divmod(i, 8)
        w = synth.philox4x32_10((g, 0, tid, synth._TAG), (seed & 0xFFFFFFFF, seed >> 32))[lane >> 1]
        h = (w >> 16) if lane & 1 else (w & 0xFFFF)
        v = np.float32(np.float32(np.float32(0.02) * Z[h]) * np.float32(0.01))
        assert t32[i].item() == v
        assert t16[i].item() == torch.tensor(v).to(torch.bfloat16).item()


def test_weights_have_the_stated_law_and_planting():
    cfg = synth.MODELS["tiny"]
    planted = synth.planted_blocks(cfg)
    assert len(planted) == 4 and len(set(planted)) == 4 and planted == synth.planted_blocks(cfg)
    b_p, b_n = planted[0], [b for b in range(cfg.n_blocks) if b not in planted][0]
    assert abs(synth.make_tensor(cfg, "wq", b_p).std().item() - 0.02) < 5e-4
    assert abs(synth.make_tensor(cfg, "wo", b_p).std().item() - 0.0002) < 5e-6
    assert abs(synth.make_tensor(cfg, "wdown", b_n).std().item() - 0.02) < 5e-4
    assert torch.equal(synth.make_tensor(cfg, "attn_norm", 0), torch.ones(cfg.d_model))
    assert not torch.equal(synth.make_tensor(cfg, "wq", 0), synth.make_tensor(cfg, "wq", 1))


def test_prompts_masks_and_patterns():
    cfg = synth.MODELS["13b"]
    p = synth.prompt(cfg, 64)
    assert len(p) == 64 and all(0 <= t < cfg.vocab for t in p) and len(set(p)) > 50
    assert len(synth.draft_blocks(cfg, 18)) == 18 and synth.draft_blocks(cfg, 18) == synth.planted_blocks(cfg)
    d20 = synth.draft_blocks(cfg, 20)
    assert len(set(d20)) == 20 and set(synth.planted_blocks(cfg)) < set(d20)
    u = synth.uniform_blocks(40, 18)
    assert len(u) == 18 and max(np.diff(u)) <= 3
    m = synth.candidate_masks(cfg, 18, 32, 0)
    assert m.shape == (32, 80) and np.all(m.sum(1) == 36) and np.all(m[:, 0::2] == m[:, 1::2])
    assert len({tuple(r) for r in m}) == 32
    assert not np.array_equal(m, synth.candidate_masks(cfg, 18, 32, 1))
