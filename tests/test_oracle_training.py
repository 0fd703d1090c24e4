"""Pins for the training oracle: the loss by hand, gradients by finite differences, and torch's own BCE-with-logits
loss, autograd and Adam on the CPU as an independent implementation."""
import math

import numpy as np
import torch

from oracle import scorer as OS
from oracle import training as OT


def _problem(seed=0, N=12, D=7, m=5):
    g = np.random.default_rng(seed)
    H = g.standard_normal((N, D)); y = (g.random(N) < 0.4).astype(np.float64); y[0], y[1] = 1.0, 0.0
    W1 = g.standard_normal((m, D)) * 0.5; b1 = g.standard_normal(m) * 0.1
    w2 = g.standard_normal(m) * 0.5; b2 = 0.2
    return H, y, W1, b1, w2, b2


def test_loss_by_hand():
    # one positive and one negative sample, scorer outputs 0.75 and 0.5 (the scorer's own hand example: y = sigmoid(ReLU(h)))
    H = np.array([[math.log(3.0)], [0.0]]); y = np.array([1.0, 0.0])
    loss, *_ = OT.loss_and_gradients(H, y, np.ones((1, 1)), np.zeros(1), np.ones(1), 0.0, alpha=2.0)
    assert abs(loss - (-(2.0 * math.log(0.75) + math.log(0.5)) / 2.0)) < 1e-12
    assert abs(OS.step_score(H[0], np.ones((1, 1)), np.zeros(1), np.ones(1), 0.0) - 0.75) < 1e-12
    assert OT.class_weight([0, 0, 0, 1, 1, 0]) == 2.0            # K- / K+ = 4 / 2


def test_gradients_by_finite_differences():
    H, y, W1, b1, w2, b2 = _problem()
    alpha = OT.class_weight(y)
    _, g_W1, g_b1, g_w2, g_b2 = OT.loss_and_gradients(H, y, W1, b1, w2, b2, alpha)
    f = lambda W1_, b1_, w2_, b2_: OT.loss_and_gradients(H, y, W1_, b1_, w2_, b2_, alpha)[0]
    eps = 1e-6
    for (i, j) in [(0, 0), (2, 3), (4, 6)]:
        d = np.zeros_like(W1); d[i, j] = eps
        assert abs((f(W1 + d, b1, w2, b2) - f(W1 - d, b1, w2, b2)) / (2 * eps) - g_W1[i, j]) < 1e-7
    for i in range(5):
        d = np.zeros(5); d[i] = eps
        assert abs((f(W1, b1 + d, w2, b2) - f(W1, b1 - d, w2, b2)) / (2 * eps) - g_b1[i]) < 1e-7
        assert abs((f(W1, b1, w2 + d, b2) - f(W1, b1, w2 - d, b2)) / (2 * eps) - g_w2[i]) < 1e-7
    assert abs((f(W1, b1, w2, b2 + eps) - f(W1, b1, w2, b2 - eps)) / (2 * eps) - g_b2) < 1e-7


def test_against_torch_loss_autograd_and_adam():
    H, y, W1, b1, w2, b2 = _problem(seed=3, N=32, D=16, m=8)
    alpha = OT.class_weight(y)
    tp = [torch.tensor(x, dtype=torch.float64, requires_grad=True) for x in (W1, b1, w2, np.array([b2]))]
    opt_t = torch.optim.Adam(tp, lr=1e-4, weight_decay=1e-5)
    lossf = torch.nn.BCEWithLogitsLoss(pos_weight=torch.tensor(alpha, dtype=torch.float64))
    params = [W1, b1, w2, np.array([b2])]
    opt_o = OT.Adam(params)
    Ht, yt = torch.tensor(H), torch.tensor(y)
    for step in range(4):
        opt_t.zero_grad()
        z = torch.relu(Ht @ tp[0].T + tp[1]) @ tp[2] + tp[3]
        lt = lossf(z, yt); lt.backward(); opt_t.step()
        lo, params = OT.train_step(H, y, params, opt_o, alpha)
        assert abs(lo - lt.item()) < 1e-12
        for a, b in zip(params, tp):
            np.testing.assert_allclose(a, b.detach().numpy(), rtol=0, atol=1e-12)


def test_training_separates_two_clusters():
    """A sanity property: on linearly separable hidden states the loss falls and the scores order the classes."""
    g = np.random.default_rng(5)
    N, D, m = 128, 16, 8
    y = (np.arange(N) % 2).astype(np.float64)
    H = g.standard_normal((N, D)) * 0.3 + np.outer(2 * y - 1, np.ones(D)) * 0.5
    params = [g.standard_normal((m, D)) * 0.1, np.zeros(m), g.standard_normal(m) * 0.1, np.zeros(1)]
    opt = OT.Adam(params, lr=1e-2, weight_decay=0.0)
    losses = []
    for _ in range(60):
        l, params = OT.train_step(H, y, params, opt, 1.0)
        losses.append(l)
    assert losses[-1] < 0.25 * losses[0]
    s = np.array([OS.step_score(h, params[0], params[1], params[2], float(params[3][0])) for h in H])
    assert s[y == 1].min() > s[y == 0].max()


def test_first_adam_step_closed_form():
    """With zero moments the first bias-corrected update is lr * g / (|g| + eps): every parameter moves by (almost)
    exactly lr against the sign of its gradient, whatever the gradient's size; weight decay enters through g."""
    p = [np.array([[0.5, -2.0]]), np.array([3.0])]
    g = [np.array([[1e-3, -40.0]]), np.array([0.0])]
    opt = OT.Adam(p, lr=1e-2, eps=1e-8, weight_decay=0.0)
    q = opt.step(p, g)
    np.testing.assert_allclose(q[0], [[0.5 - 1e-2 * 1e-3 / (1e-3 + 1e-8), -2.0 + 1e-2 * 40.0 / (40.0 + 1e-8)]], rtol=0, atol=1e-15)
    assert q[1][0] == 3.0                                             # zero gradient, no decay: no move
    opt = OT.Adam(p, lr=1e-2, eps=1e-8, weight_decay=0.1)
    q = opt.step(p, g)
    g_eff = 0.0 + 0.1 * 3.0                                           # decay times the parameter joins the gradient
    assert abs(q[1][0] - (3.0 - 1e-2 * g_eff / (g_eff + 1e-8))) < 1e-15
    # second step from the same gradient: m = (1 - b1^2) g / (1 - b1^2) = g, v likewise -> the same step again
    r = OT.Adam([np.array([1.0])], lr=1e-3, weight_decay=0.0)
    a = r.step([np.array([1.0])], [np.array([2.0])])
    b = r.step(a, [np.array([2.0])])
    assert abs((a[0][0] - 1.0) - (b[0][0] - a[0][0])) < 1e-12
