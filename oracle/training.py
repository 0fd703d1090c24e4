"""Oracle: one optimisation step of the step scorer (fp64).

TEST INFRASTRUCTURE ONLY - never imported by the product path.

Sec. 3.1 "Training Objective": weighted binary cross-entropy over the N steps of a batch,

    L = -(1/N) sum_n ( alpha * y_n * log yhat_n + (1 - y_n) * log(1 - yhat_n) ),   alpha = K- / K+,

with yhat = sigmoid(w2 . ReLU(W1 h + b1) + b2) (the scorer of scorer.py).  The appendix "Training Parameters" fixes
batch 128, Adam, learning rate 1e-4, weight decay 1e-5 and a loss computed from logits.

Readings where the paper is silent: Adam's beta1 = 0.9, beta2 = 0.999, eps = 1e-8 (the optimiser's customary
defaults); "weight decay" with Adam is the L2 form (the decay times the parameter is added to the gradient before
the moments are updated) and applies to every parameter; the ReLU's derivative at exactly 0 is 0.
"""
from __future__ import annotations

import numpy as np


def class_weight(labels) -> float:
    """alpha = K- / K+ : negative over positive samples."""
    labels = np.asarray(labels)
    return float(np.sum(labels == 0)) / float(np.sum(labels == 1))


def loss_and_gradients(H, y, W1, b1, w2, b2, alpha):
    """Loss of the batch and its gradients with respect to W1, b1, w2, b2 (all float64)."""
    H, y = np.asarray(H, dtype=np.float64), np.asarray(y, dtype=np.float64)
    W1, b1, w2 = (np.asarray(x, dtype=np.float64) for x in (W1, b1, w2))
    N = H.shape[0]
    pre = H @ W1.T + b1
    a = np.where(pre > 0.0, pre, 0.0)
    z = a @ w2 + float(b2)
    # log sigmoid(z) and log(1 - sigmoid(z)) without overflow
    log_sig = -np.logaddexp(0.0, -z)
    log_one_minus = -np.logaddexp(0.0, z)
    loss = -np.mean(alpha * y * log_sig + (1.0 - y) * log_one_minus)
    sig = 1.0 / (1.0 + np.exp(-z))
    dz = ((1.0 - y) * sig - alpha * y * (1.0 - sig)) / N
    g_w2 = a.T @ dz
    g_b2 = float(np.sum(dz))
    dpre = np.outer(dz, w2) * (pre > 0.0)
    g_b1 = dpre.sum(axis=0)
    g_W1 = dpre.T @ H
    return float(loss), g_W1, g_b1, g_w2, g_b2


class Adam:
    """Adam with the weight decay added to the gradient, one state per parameter array."""

    def __init__(self, params, lr=1e-4, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-5):
        self.lr, self.beta1, self.beta2, self.eps, self.wd = lr, beta1, beta2, eps, weight_decay
        self.m = [np.zeros_like(np.asarray(p, dtype=np.float64)) for p in params]
        self.v = [np.zeros_like(x) for x in self.m]
        self.t = 0

    def step(self, params, grads):
        self.t += 1
        out = []
        for i, (p, g) in enumerate(zip(params, grads)):
            p = np.asarray(p, dtype=np.float64)
            g = np.asarray(g, dtype=np.float64) + self.wd * p
            self.m[i] = self.beta1 * self.m[i] + (1.0 - self.beta1) * g
            self.v[i] = self.beta2 * self.v[i] + (1.0 - self.beta2) * g * g
            m_hat = self.m[i] / (1.0 - self.beta1 ** self.t)
            v_hat = self.v[i] / (1.0 - self.beta2 ** self.t)
            out.append(p - self.lr * m_hat / (np.sqrt(v_hat) + self.eps))
        return out


def train_step(H, y, params, opt: Adam, alpha):
    """params = [W1, b1, w2, b2 (shape (1,))].  Returns (loss before the update, new params)."""
    W1, b1, w2, b2 = params
    loss, g_W1, g_b1, g_w2, g_b2 = loss_and_gradients(H, y, W1, b1, w2, float(np.asarray(b2).reshape(-1)[0]), alpha)
    return loss, opt.step([W1, b1, w2, np.asarray(b2, dtype=np.float64).reshape(1)], [g_W1, g_b1, g_w2, np.array([g_b2])])
