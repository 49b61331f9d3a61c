"""Training objective of the retaining head (Eq. 2, Eq. 3) on the GPU against the oracle."""

import numpy as np
import pytest
import torch

import workloads as W
from oracle import locret_oracle as O

pytestmark = pytest.mark.gpu


def case(n, d_in, d_R, hk, seed):
    g = np.random.default_rng(7000 + seed)
    z = W.to_bf16_grid(g.standard_normal((n, d_in)).astype(np.float32))
    w1 = W.to_bf16_grid((g.standard_normal((d_in, d_R)) / np.sqrt(d_in)).astype(np.float32))
    w2 = W.to_bf16_grid((g.standard_normal((d_R, hk)) / np.sqrt(d_R)).astype(np.float32))
    labels = (g.standard_normal((hk, n)) * 1.5).astype(np.float32)      # errors on both sides of the Smooth-L1 knee
    return z, w1, w2, labels


@pytest.mark.parametrize("n,d_in,d_R,hk", [(128, 128, 64, 2), (1024, 768, 256, 2), (2048, 6144, 1024, 8)])
def test_loss_and_gradients_match_the_oracle(n, d_in, d_R, hk):
    from parity_util import bf16_dev
    from paper_2410_01805_b200 import rh_loss_grad
    z, w1, w2, labels = case(n, d_in, d_R, hk, n)
    alpha = 0.05
    loss, dw1, dw2 = O.rh_loss_and_grads(z, labels, w1, w2, alpha)
    gl, g1, g2 = rh_loss_grad(bf16_dev(z), torch.from_numpy(labels).cuda(), bf16_dev(w1), bf16_dev(w2), alpha)
    gl, g1, g2 = float(gl.item()), g1.cpu().numpy().astype(np.float64), g2.cpu().numpy().astype(np.float64)
    # loss and dW2 come from fp32 arithmetic on exact bf16 products: only summation order differs
    assert abs(gl - loss) <= 1e-4 * abs(loss)
    assert np.abs(g2 - dw2).max() <= 1e-4 * np.abs(dw2).max()
    # dW1 = z^T dpre with dpre rounded to bf16 for the contraction: every term carries at most 2^-9
    # relative error, so |Δ| <= 2^-8 (|z|^T |dpre|) element-wise (twice the worst case, for the fp32 sums)
    zf = np.asarray(z, np.float64)
    pre = zf @ np.asarray(w1, np.float64)
    sig = 1.0 / (1.0 + np.exp(-pre))
    s = (pre * sig) @ np.asarray(w2, np.float64)
    ds = np.clip(s - labels.T.astype(np.float64), -1.0, 1.0)
    adj = s[:-1] - s[1:]
    ds[:-1] += 2 * alpha * adj
    ds[1:] -= 2 * alpha * adj
    dpre = (ds @ np.asarray(w2, np.float64).T) * (sig * (1.0 + pre * (1.0 - sig)))
    bound = 2.0 ** -8 * (np.abs(zf).T @ np.abs(dpre)) + 1e-6
    assert (np.abs(g1 - dw1) <= bound).all(), float((np.abs(g1 - dw1) / bound).max())
    # and in practice the errors are random: far inside the worst case
    assert np.abs(g1 - dw1).max() <= 2e-2 * np.sqrt(np.mean(dw1 ** 2))


def test_training_argument_checks():
    from paper_2410_01805_b200 import LocretError, rh_loss_grad
    z = torch.zeros((100, 128), dtype=torch.bfloat16, device="cuda")          # n not a multiple of 64
    w1 = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
    w2 = torch.zeros((64, 2), dtype=torch.bfloat16, device="cuda")
    lab = torch.zeros((2, 100), dtype=torch.float32, device="cuda")
    with pytest.raises(LocretError):
        rh_loss_grad(z, lab, w1, w2)


def test_adamw_step_matches_the_oracle_on_seeded_inputs():
    """The optimiser kernel alone: parameters, gradients and moments come from the seeded generator
    (nothing the CUDA path computed goes into the oracle)."""
    from paper_2410_01805_b200 import adamw_step
    g = np.random.default_rng(8000)
    n = 100_003
    p = g.standard_normal(n).astype(np.float32)
    gr = (g.standard_normal(n) * 0.1).astype(np.float32)
    m = (g.standard_normal(n) * 0.01).astype(np.float32)
    v = (g.random(n) * 1e-3).astype(np.float32)
    for step, lr in ((1, 5e-4), (7, 2e-2)):
        rp, rm, rv = O.adamw_step(p, gr, m, v, step, lr)
        P, G, M, V = (torch.from_numpy(a.copy()).cuda() for a in (p, gr, m, v))
        B = torch.zeros(n, dtype=torch.bfloat16, device="cuda")
        adamw_step(P, G, M, V, step, lr, param_bf16=B)
        torch.cuda.synchronize()
        assert np.abs(P.cpu().numpy() - rp).max() <= 1e-6 * max(1.0, np.abs(rp).max())
        assert np.abs(M.cpu().numpy() - rm).max() <= 1e-7 and np.abs(V.cpu().numpy() - rv).max() <= 1e-8
        assert torch.equal(B, P.to(torch.bfloat16))


def test_a_few_training_steps_follow_the_oracle_and_reduce_the_loss():
    """Labels from the definition, loss and gradients, AdamW: three updates, each side on its OWN
    trajectory (the oracle's fp64 master weights and moments are updated with the oracle's own
    gradients; nothing the CUDA path computed is fed to it).  Both compute the forward pass from the
    bf16 rounding of their master weights.  The first Adam updates have magnitude lr whatever the
    gradient's size, so an element whose gradient is smaller than the gradient error may move the other
    way on the two sides: parameters are compared where the oracle's gradient is well above that error."""
    from parity_util import bf16_dev
    from paper_2410_01805_b200 import adamw_step, cis_labels, rh_loss_grad
    g = np.random.default_rng(8100)
    n, h, hk, d, d_R, n_a = 512, 4, 2, 64, 128, 64
    d_in = (h + 2 * hk) * d
    qkv = W.to_bf16_grid(g.standard_normal((n + n_a, d_in)).astype(np.float32))
    q = qkv[:, : h * d].reshape(n + n_a, h, d)
    k = qkv[:, h * d:(h + hk) * d].reshape(n + n_a, hk, d)
    labels = cis_labels(bf16_dev(np.ascontiguousarray(q[n:])), bf16_dev(np.ascontiguousarray(k[:n])), 1.0 / np.sqrt(d))
    ref_labels = O.cis_labels(q[n:], k[:n], hk, 1.0 / np.sqrt(d))
    assert np.abs(labels.cpu().numpy() - ref_labels).max() < 1e-4 * max(1.0, np.abs(ref_labels).max())
    z = qkv[:n]
    w1 = (g.standard_normal((d_in, d_R)) / np.sqrt(d_in)).astype(np.float32)
    w2 = (g.standard_normal((d_R, hk)) / np.sqrt(d_R)).astype(np.float32)
    P1, P2 = torch.from_numpy(w1).cuda(), torch.from_numpy(w2).cuda()
    B1, B2 = P1.to(torch.bfloat16), P2.to(torch.bfloat16)
    M1, V1, M2, V2 = (torch.zeros_like(t) for t in (P1, P1, P2, P2))
    o1, o2 = w1.astype(np.float64), w2.astype(np.float64)
    om1, ov1, om2, ov2 = (np.zeros_like(a) for a in (o1, o1, o2, o2))
    zd = bf16_dev(z)
    losses, ref_losses = [], []
    lr = 2e-2
    sure1 = np.ones_like(o1, dtype=bool)
    sure2 = np.ones_like(o2, dtype=bool)
    for step in range(1, 4):
        loss, g1, g2 = rh_loss_grad(zd, labels, B1, B2, 2.5e-3)
        rl, r1, r2 = O.rh_loss_and_grads(z, ref_labels, O.round_bf16(o1), O.round_bf16(o2), 2.5e-3)
        losses.append(float(loss.item())); ref_losses.append(rl)
        tol = 1e-3 if step == 1 else 5e-2          # later steps: the trajectories have parted on the unsure elements
        assert abs(losses[-1] - rl) <= tol * abs(rl), (step, losses[-1], rl)
        if step == 1:
            assert np.abs(g2.cpu().numpy() - r2).max() <= 1e-3 * np.abs(r2).max()
            assert np.abs(g1.cpu().numpy() - r1).max() <= 2e-2 * np.sqrt(np.mean(r1 ** 2))
        sure1 &= np.abs(r1) > 0.2 * np.sqrt(np.mean(r1 ** 2))
        sure2 &= np.abs(r2) > 0.2 * np.sqrt(np.mean(r2 ** 2))
        o1, om1, ov1 = O.adamw_step(o1, r1, om1, ov1, step, lr)
        o2, om2, ov2 = O.adamw_step(o2, r2, om2, ov2, step, lr)
        adamw_step(P1, g1, M1, V1, step, lr, param_bf16=B1)
        adamw_step(P2, g2, M2, V2, step, lr, param_bf16=B2)
        torch.cuda.synchronize()
        assert torch.equal(B1, P1.to(torch.bfloat16))
    assert sure1.mean() > 0.2 and sure2.mean() > 0.2      # (a third of the elements stay clear of zero gradient in all three steps)
    assert np.abs(P1.cpu().numpy() - o1)[sure1].max() <= 0.25 * lr
    assert np.abs(P2.cpu().numpy() - o2)[sure2].max() <= 0.25 * lr
    assert losses[2] < losses[0] and ref_losses[2] < ref_losses[0]
