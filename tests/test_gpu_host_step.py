"""aa_step_host: the whole step for callers whose pool, Boss logits and labels live in host memory.

The call copies the inputs to its device staging buffer, screens the pool (Algorithm 1), takes the losses of the
accepted instances from the first M logit rows, updates the linear Assistant (Algorithm 2) and copies back the batch
list, its count and the losses.  Bars as in test_gpu_parity.py: list bit-exact outside the tie band |p - c| < 1e-5,
losses abs 1e-4, parameters rel 1e-4 (+ 1e-4 rms floor).
"""
import math

import numpy as np
import pytest
import torch

from oracle import aa_oracle as O
from paper_1905_03381_b200 import binding as B
from paper_1905_03381_b200 import build, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def params_close(got, ref):
    ref = np.asarray(ref, np.float64).reshape(-1)
    got = np.asarray(got, np.float64).reshape(-1)
    tol = 1e-4 * np.abs(ref) + 1e-4 * math.sqrt(float(np.mean(ref ** 2)) + 1e-300)
    assert np.all(np.abs(got - ref) <= tol), float(np.max(np.abs(got - ref) - tol))


@pytest.mark.parametrize("n,d,classes,dtype,mix,lr,thr", [
    (5000, 256, 10, torch.bfloat16, 0.2, 0.1, None), (3001, 64, 7, torch.float32, 0.1, 0.05, 1.2),
    (20000, 3072, 100, torch.bfloat16, 0.1, 0.05, None),
])
def test_host_step_matches_the_oracle(n, d, classes, dtype, mix, lr, thr):
    build.build()
    x = W.normal((n, d), 1.0, 400 + n, dtype, "cpu").pin_memory()
    logits = W.normal((n, classes), 2.0, 401 + n, torch.float32, "cpu").pin_memory()
    labels = W.randint(0, classes, (n,), 402 + n, "cpu").pin_memory()
    w0, b0 = W.linear_assistant(d, 403, DEV)
    w0 = (w0 * 30.0).contiguous()                       # scores spread enough for both labels to occur
    w, b = w0.clone(), b0.clone()
    out_idx = torch.full((n,), -7, dtype=torch.int32).pin_memory()
    out_count = torch.full((1,), -7, dtype=torch.int32).pin_memory()
    out_loss = torch.full((n,), -7.0, dtype=torch.float32).pin_memory()
    aa = B.AutoAssist(max_rows=n, max_d=d, device=DEV)
    feat, lg, staging, nbytes = aa.host_step_plan(x, logits)
    seed, step = 11, 3
    aa.aa_step_host(feat, B.linear_assistant(w, b), mix, seed, step, lg, labels, lr, out_idx, out_count, out_loss,
                    staging, nbytes, threshold=thr)
    assert aa.aa_device_status() == B.AA_OK
    m = int(out_count.item())
    idx = out_idx.numpy()[:m].astype(np.int64)
    assert 0 < m < n and np.all(np.diff(idx) > 0)
    assert np.all(out_idx.numpy()[m:] == -7) and np.all(out_loss.numpy()[m:] == -7.0)     # nothing else comes back
    # screening: the oracle's decisions on the same pool; outside the tie band the batch is the oracle's batch
    xo = W.to_oracle(x)
    w_h, b_h = w0.cpu().numpy(), float(b0.item())
    s_ref = O.score_dense(xo, w_h, b_h)
    g = O.sigmoid(s_ref)
    keep = O.shrink(g, mix, seed, step)
    far = np.abs(O.accept_prob(g, mix) - O.uniform(seed, step, np.arange(n))) >= 1e-5
    got = np.zeros(n, np.uint8)
    got[idx] = 1
    assert np.array_equal(got[far], keep[far])
    # losses: row k of the logits is the Boss's output for the k-th accepted instance
    f_ref = O.row_loss(logits.numpy()[:m], labels.numpy()[:m])
    f_gpu = out_loss.numpy()[:m]
    assert np.max(np.abs(f_gpu - f_ref)) <= 1e-4
    # update: Algorithm 2 on the batch the GPU took, with the losses it returned
    w_ref, b_ref, z = O.assistant_step_linear_dense(xo, f_gpu, w_h, b_h, lr, T=thr, row_idx=idx.astype(np.int32))
    assert 0 < z.sum() < m
    params_close(w.cpu().numpy(), w_ref)
    params_close([b.item()], [b_ref])
    assert float((w - w0).abs().max()) > 0
    aa.close()


def test_host_step_rejects_what_it_cannot_take():
    build.build()
    n, d = 64, 32
    x = torch.zeros((n, d), dtype=torch.float32).pin_memory()
    logits = torch.zeros((n, 4), dtype=torch.float32).pin_memory()
    labels = torch.zeros(n, dtype=torch.int32).pin_memory()
    w, b = torch.zeros(d, device=DEV), torch.zeros(1, device=DEV)
    out_idx, out_count, out_loss = torch.zeros(n, dtype=torch.int32), torch.zeros(1, dtype=torch.int32), torch.zeros(n)
    aa = B.AutoAssist(max_rows=n, max_d=d, device=DEV)
    feat, lg, staging, nbytes = aa.host_step_plan(x, logits)
    with pytest.raises(B.AutoAssistError):      # a staging buffer that is too small
        aa.aa_step_host(feat, B.linear_assistant(w, b), 0.1, 0, 0, lg, labels, 0.1, out_idx, out_count, out_loss, staging, nbytes // 2)
    # mix = 1 keeps every instance: the batch is the pool, in order
    aa.aa_step_host(feat, B.linear_assistant(w, b), 1.0, 0, 0, lg, labels, 0.1, out_idx, out_count, out_loss, staging, nbytes)
    assert int(out_count.item()) == n and np.array_equal(out_idx.numpy(), np.arange(n))
    assert np.max(np.abs(out_loss.numpy() - math.log(4.0))) <= 1e-5      # uniform logits: ln C
    assert aa.aa_device_status() == B.AA_OK
    aa.close()
