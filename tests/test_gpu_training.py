"""scorer_train_step against the training oracle: loss and parameters over several Adam steps."""
import numpy as np
import pytest
import torch

from oracle import training as OT
from paper_2601_09093_b200 import binding as B

pytestmark = pytest.mark.gpu


def _case(seed, N, D, m, dtype):
    g = np.random.default_rng(seed)
    y = (g.random(N) < 0.3).astype(np.float64); y[0] = 1.0
    if N > 1:
        y[1] = 0.0
    H = g.standard_normal((N, D)) + np.outer(2 * y - 1, g.standard_normal(D) * 0.2)
    Ht = torch.tensor(H, dtype=dtype)
    H = Ht.double().numpy()                          # the oracle sees the rounded hidden states
    W1 = (g.standard_normal((m, D)) / np.sqrt(D)).astype(np.float32)
    b1 = (g.standard_normal(m) * 0.05).astype(np.float32)
    w2 = (g.standard_normal(m) / np.sqrt(m)).astype(np.float32)
    b2 = np.float32(0.1)
    return H, Ht, y, W1, b1, w2, b2


@pytest.mark.parametrize("N,D,m,dtype,steps", [
    (128, 4096, 512, torch.bfloat16, 5),             # the paper's batch on the 4B model's scorer
    (128, 1024, 256, torch.float32, 5),
    (37, 200, 70, torch.float32, 8),                 # ragged in every dimension
    (1, 64, 8, torch.bfloat16, 3),
    (300, 520, 130, torch.bfloat16, 4),
])
def test_train_step_matches_oracle(N, D, m, dtype, steps):
    H, Ht, y, W1, b1, w2, b2 = _case(11 + N, N, D, m, dtype)
    alpha = OT.class_weight(y) if N > 1 else 1.0
    dev = "cuda:0"
    tr = B.ScorerTrainer(torch.tensor(W1, device=dev), torch.tensor(b1, device=dev), torch.tensor(w2, device=dev),
                         float(b2), batch=N, pos_weight=alpha)
    params = [W1.astype(np.float64), b1.astype(np.float64), w2.astype(np.float64), np.array([float(b2)])]
    opt = OT.Adam(params)
    Hd = Ht.to(dev); yd = torch.tensor(y, dtype=torch.float32, device=dev)
    for _ in range(steps):
        loss_gpu = float(tr.step(Hd, yd).cpu()[0])
        loss_ref, params = OT.train_step(H, y, params, opt, alpha)
        assert abs(loss_gpu - loss_ref) <= 2e-5 * max(1.0, abs(loss_ref))
    torch.cuda.synchronize()
    # every step moves a parameter by about lr = 1e-4; the fp32 path must follow the fp64 one to a few percent of one step
    for ref, got in zip(params, (tr.W1, tr.b1, tr.w2, tr.b2)):
        np.testing.assert_allclose(got.cpu().numpy().reshape(ref.shape), ref, rtol=0, atol=5e-6)
    moved = np.abs(tr.W1.cpu().numpy() - W1).max()
    assert moved > 0.5e-4 * steps                    # the update happened


def test_train_step_rejects_bad_arguments():
    dev = "cuda:0"
    tr = B.ScorerTrainer(torch.zeros(8, 64, device=dev), torch.zeros(8, device=dev), torch.zeros(8, device=dev), 0.0, batch=4)
    h = torch.zeros(4, 64, device=dev); y = torch.zeros(4, device=dev)
    rc = B.lib().scorer_train_step(B._ptr(h), B.STEP_FP32, B._ptr(y), 4, B._ptr(tr.W1), B._ptr(tr.b1), B._ptr(tr.w2),
                                   B._ptr(tr.b2), 64, 8, B._ptr(tr.adam_m), B._ptr(tr.adam_v), B.C.byref(tr.h),
                                   B._ptr(tr.ws), tr.ws_bytes, B._ptr(tr.loss), None)
    assert rc != 0                                   # step 0: the caller has to count from 1
    tr.h.step = 1
    rc = B.lib().scorer_train_step(B._ptr(h), B.STEP_FP32, B._ptr(y), 4, B._ptr(tr.W1), B._ptr(tr.b1), B._ptr(tr.w2),
                                   B._ptr(tr.b2), 64, 8, B._ptr(tr.adam_m), B._ptr(tr.adam_v), B.C.byref(tr.h),
                                   B._ptr(tr.ws), tr.ws_bytes - 256, B._ptr(tr.loss), None)
    assert rc != 0                                   # workspace too small
