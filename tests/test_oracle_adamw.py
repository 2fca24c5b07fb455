"""Pins for the oracle's AdamW step on the DeltaBuffer: PyTorch's CPU AdamW (an independent implementation,
different operation order, so a tolerance), the closed form of the first step, and weight-decay-only motion."""
import numpy as np
import torch

from oracle import falqon_oracle as orc


def test_matches_library_adamw_over_several_steps():
    rng = np.random.default_rng(0)
    shape = (37, 16)
    p0 = (rng.standard_normal(shape) * 1e-3).astype(np.float32)
    hp = dict(lr=2e-4, betas=(0.9, 0.999), eps=1e-8, weight_decay=0.01)
    tp = torch.nn.Parameter(torch.from_numpy(p0.copy()))
    opt = torch.optim.AdamW([tp], **hp)
    p, m, v = p0.copy(), np.zeros(shape, np.float32), np.zeros(shape, np.float32)
    for step in range(1, 8):
        g = (rng.standard_normal(shape) * 10.0 ** rng.integers(-6, 0)).astype(np.float32)
        tp.grad = torch.from_numpy(g.copy())
        opt.step()
        orc.adamw_step(p, g, m, v, hp["lr"], 0.9, 0.999, hp["eps"], hp["weight_decay"], step)
        ref = tp.detach().numpy()
        # the library keeps beta2 in double (1 - 0.999 = 1.0000e-3); here it is the fp32 value (1 - 0.99900001 =
        # 0.99999e-3): 1.3e-5 relative on v, half of that on the update
        assert np.allclose(p, ref, rtol=5e-5, atol=1e-9), step
        st = opt.state[tp]
        assert np.allclose(m, st["exp_avg"].numpy(), rtol=5e-5, atol=1e-9)   # sign changes cancel: compare absolutely too
        assert np.allclose(v, st["exp_avg_sq"].numpy(), rtol=5e-5, atol=1e-20)


def test_first_step_closed_form_and_decay_only():
    g = np.array([[3.0, -0.5, 1e-3, 0.0]], dtype=np.float32)
    p = np.zeros((1, 4), np.float32); m = np.zeros_like(p); v = np.zeros_like(p)
    orc.adamw_step(p, g, m, v, 1e-2, 0.9, 0.999, 0.0, 0.0, 1)
    # t = 1: m_hat = g, v_hat = g^2  ->  the update is lr * sign(g); a zero gradient divides 0 by 0 without eps
    assert np.allclose(p[0, :3], -1e-2 * np.sign(g[0, :3]), rtol=1e-5) and np.isnan(p[0, 3])
    p = np.full((2, 2), 4.0, np.float32); m = np.zeros_like(p); v = np.zeros_like(p)
    orc.adamw_step(p, np.zeros_like(p), m, v, 0.5, 0.9, 0.999, 1e-8, 0.1, 3)
    assert np.all(p == np.float32(4.0) * np.float32(1 - 0.5 * 0.1)) and not m.any() and not v.any()
