"""The seeded input generator: integer recipe checked against big-int Python, and distribution shape."""
import numpy as np
import torch

from paper_2510_24061_b200 import synth


def test_normal_matches_bigint_recipe():
    x = synth.normal_bf16(3, synth.TID_W + 16, (257, 33), 0.02)
    key = synth.tensor_key(3, synth.TID_W + 16)
    for i in [0, 1, 32, 33, 4097, 257 * 33 - 1]:
        total = 0
        for d in range(3):
            w = synth._mix64_i(key + (3 * i + d + 1) * synth._GOLD)
            total += sum((w >> (16 * f)) & 0xFFFF for f in range(4))
        z = np.float32((total - 393210) * 2.0 ** -16)
        want = torch.tensor(z * np.float32(0.02)).to(torch.bfloat16)
        assert x.flatten()[i] == want


def test_distributions_and_determinism():
    x = synth.normal_bf16(0, 0, (512, 1024), 1.0).float()
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01 and x.abs().max() <= 6.0
    u = synth.uniform_bf16(0, 2, (64, 1024), 1 / 32).float()
    assert u.min() >= -1 / 32 and u.max() <= 1 / 32 and abs(u.mean()) < 1e-3
    assert abs(u.std() - (1 / 32) / 3 ** 0.5) < 5e-4
    assert torch.equal(synth.normal_bf16(0, 0, (512, 1024), 1.0).float(), x)
    assert not torch.equal(synth.normal_bf16(1, 0, (512, 1024), 1.0).float(), x)
    t = synth.student_t3_bf16(0, 1, (256, 1024), 0.02).float()
    assert t.abs().max() > 0.02 * 8  # heavy tails


def test_activation_outlier_channels():
    cfg = synth.config0()
    x = synth.activations(cfg["seed"], 0, cfg["T"], cfg["n"], cfg["n_outliers"]).float()
    cols = synth.outlier_columns(cfg["n"], cfg["n_outliers"])
    assert cols == [0, 128, 256, 384, 512, 640, 768, 896]
    ratio = x[:, cols].std() / x[:, [c + 1 for c in cols]].std()
    assert 14 < ratio < 18


def test_projection_shapes_give_the_papers_parameter_counts():
    """Rank 64 on all seven projections of every block: the DeltaBuffers (B only) of the 7B shapes hold 87.0 M values, A
    and B together 159.9 M (the paper's table rounds these to 80 M and 160 M), and 250.3 M for the 13B shapes (250 M)."""
    from paper_2510_24061_b200 import synth
    r = 64
    b7 = 32 * sum(m * r for _, n, m in synth.LLAMA_7B_LINEARS)
    ab7 = 32 * sum((m + n) * r for _, n, m in synth.LLAMA_7B_LINEARS)
    ab13 = 40 * sum((m + n) * r for _, n, m in synth.LLAMA_13B_LINEARS)
    assert round(b7 / 1e6, 1) == 87.0 and round(ab7 / 1e6, 1) == 159.9 and round(ab13 / 1e6, 1) == 250.3
    assert abs(ab7 / 160e6 - 1) < 0.01 and abs(ab13 / 250e6 - 1) < 0.01
    # backbone bytes of the 7B stack in FP8: 6.48 GB
    assert round(32 * sum(m * n for _, n, m in synth.LLAMA_7B_LINEARS) / 1e9, 2) == 6.48
