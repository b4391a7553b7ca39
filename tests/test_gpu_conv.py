"""The convolutional Assistant (Boss's convolution -> rectifier -> average pooling -> single linear layer): parity of the
feature kernel with the CPU oracle, and of a whole screen + update step whose linear layer runs on those features.

Bars: features |phi - phi_ref| <= 1e-5 (|phi_ref| + scale), scale = the mean over the window of |bias| + sum |tap| |pixel|
(fp32 accumulation of up to 75 products per output against fp64); the linear layer on phi is held to the bars of
test_gpu_parity.py, with the oracle given the GPU's own fp32 features (the layer's contract starts at its input).
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


@pytest.fixture(scope="module")
def aa():
    build.build()
    ctx = B.AutoAssist(max_rows=1 << 16, max_d=4096, device=DEV)
    yield ctx
    torch.cuda.synchronize()
    assert ctx.aa_device_status() == B.AA_OK
    ctx.close()


def features(aa, x, weight, bias, H, Wd, pool):
    c_out = weight.shape[0]
    F = c_out * (H // pool) * (Wd // pool)
    phi = torch.full((x.shape[0], F), -9.0, dtype=torch.float32, device=DEV)
    aa.aa_conv_pool_features(B.dense_features(x), B.conv_layer(weight, bias, H, Wd, pool), phi)
    torch.cuda.synchronize()
    return phi


@pytest.mark.parametrize("n,c_in,H,Wd,c_out,k,pool,dtype,pad", [
    (37, 3, 32, 32, 16, 3, 4, torch.bfloat16, 0), (5, 3, 32, 32, 16, 3, 32, torch.bfloat16, 0), (9, 1, 28, 28, 8, 5, 2, torch.float32, 0),
    (20, 3, 12, 12, 5, 3, 1, torch.float32, 4), (3, 2, 8, 24, 7, 1, 8, torch.bfloat16, 8), (300, 3, 32, 32, 16, 3, 8, torch.bfloat16, 0),
    (1, 3, 32, 32, 32, 3, 2, torch.float32, 0),
    # bf16 shapes of the matrix-instruction kernel: one and two k-steps, one and two channel tiles, every pooling side,
    # 1 x 1 / 3 x 3 / 5 x 5 windows, padded rows, channel counts that are not a multiple of 8
    (33, 3, 32, 32, 16, 3, 1, torch.bfloat16, 0), (21, 3, 32, 32, 16, 3, 2, torch.bfloat16, 8), (18, 3, 32, 32, 16, 3, 16, torch.bfloat16, 0),
    (40, 1, 16, 48, 5, 3, 4, torch.bfloat16, 0), (12, 1, 20, 16, 8, 5, 2, torch.bfloat16, 0), (7, 3, 8, 64, 13, 1, 8, torch.bfloat16, 16),
    (700, 3, 32, 32, 16, 3, 4, torch.bfloat16, 0),
])
def test_conv_pool_features_match_the_oracle(aa, n, c_in, H, Wd, c_out, k, pool, dtype, pad):
    d = c_in * H * Wd
    buf = W.normal((n, d + pad), 1.0, 300 + n + d, dtype, DEV)
    x = buf[:, :d]
    weight = W.normal((c_out, c_in, k, k), math.sqrt(2.0 / (c_in * k * k)), 301 + c_out, torch.float32, DEV)
    bias = W.normal((c_out,), 0.2, 302, torch.float32, DEV)
    phi = features(aa, x, weight, bias, H, Wd, pool).cpu().numpy()
    xh = W.to_oracle(x.contiguous())
    ref = O.conv_pool_features(xh, c_in, H, Wd, weight.cpu().numpy(), bias.cpu().numpy(), pool)
    # scale of the terms an output adds up: the same map with |taps|, |bias| and |pixels| (no rectifier needed: all terms >= 0)
    x_abs = x.contiguous().abs()
    scale = O.conv_pool_features(W.to_oracle(x_abs), c_in, H, Wd, weight.abs().cpu().numpy(), bias.abs().cpu().numpy(), pool)
    err = np.abs(phi - ref)
    assert np.all(err <= 1e-5 * (np.abs(ref) + scale) + 1e-30), float(np.max(err / (np.abs(ref) + scale + 1e-30)))
    assert ref.std() > 0.01


def test_identity_taps_and_global_pooling_reduce_to_the_linear_assistant_on_pooled_pixels(aa):
    n, c_in, H, Wd = 2000, 3, 32, 32
    x = W.uniform01((n, c_in * H * Wd), 310, torch.bfloat16, DEV)               # non-negative pixels: the rectifier is inert
    ident = torch.zeros((c_in, c_in, 3, 3), device=DEV)
    ident[torch.arange(c_in), torch.arange(c_in), 1, 1] = 1.0
    phi = features(aa, x, ident, None, H, Wd, 32)
    pooled = x.float().double().reshape(n, c_in, -1).mean(dim=2).cpu().numpy()
    assert np.max(np.abs(phi.cpu().numpy() - pooled)) <= 1e-5 * (pooled.max() + 1)


def test_whole_step_of_the_convolutional_assistant(aa):
    """Screen a pool with conv -> pool -> linear, then one update of the linear layer on the accepted instances."""
    n, c_in, H, Wd, c_out, pool = 3000, 3, 32, 32, 16, 4
    x = W.uniform01((n, c_in * H * Wd), 320, torch.bfloat16, DEV)
    weight = W.normal((c_out, c_in, 3, 3), math.sqrt(2.0 / 27.0), 321, torch.float32, DEV)
    bias = W.normal((c_out,), 0.1, 322, torch.float32, DEV)
    phi = features(aa, x, weight, bias, H, Wd, pool)
    F = phi.shape[1]
    ref_phi = O.conv_pool_features(W.to_oracle(x), c_in, H, Wd, weight.cpu().numpy(), bias.cpu().numpy(), pool)
    assert np.max(np.abs(phi.cpu().numpy() - ref_phi)) <= 1e-5 * (np.abs(ref_phi).max() + 1) * 10
    w = W.normal((F,), 0.05, 323, torch.float32, DEV)
    b = torch.full((1,), -0.1, device=DEV)
    asst = B.linear_assistant(w, b)
    out_idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    score = torch.zeros(n, dtype=torch.float32, device=DEV)
    mask = torch.zeros(n, dtype=torch.uint8, device=DEV)
    aa.aa_score_shrink(B.dense_features(phi), asst, 0.1, 4, 2, out_idx, cnt, score, mask)
    torch.cuda.synchronize()
    m = int(cnt.item())
    phi_h, wh = phi.cpu().numpy(), w.cpu().numpy()
    ref = O.screen_linear_dense(phi_h, wh, -0.1, 0.1, 4, 2)
    pn = np.linalg.norm(phi_h.astype(np.float64), axis=1)
    assert np.all(np.abs(score.cpu().numpy() - ref["s"]) <= 1e-5 * (np.abs(ref["s"]) + np.linalg.norm(wh) * pn))
    c = O.uniform(4, 2, np.arange(n))
    far = np.abs(ref["p"] - c) >= 1e-5
    mk = mask.cpu().numpy()
    assert np.array_equal(mk[far], ref["keep"][far])
    assert m == int(mk.sum()) and np.array_equal(out_idx.cpu().numpy()[:m], O.compact(mk))
    # and against the oracle's own features end to end: decisions agree wherever p is not within 1e-4 of the draw
    ref2 = O.screen_linear_dense(ref_phi.astype(np.float32), wh, -0.1, 0.1, 4, 2)
    far2 = np.abs(ref2["p"] - c) >= 1e-4
    assert np.array_equal(mk[far2], ref2["keep"][far2])
    loss = (W.normal((n,), 1.0, 324, torch.float32, DEV).abs() * 2).contiguous()
    w0 = wh.copy()
    aa.aa_assistant_step(B.dense_features(phi, row_idx=out_idx), loss, asst, 0.1, count_dev=cnt)
    torch.cuda.synchronize()
    rows = out_idx.cpu().numpy()[:m].astype(np.int32)
    w_ref, b_ref, z = O.assistant_step_linear_dense(phi_h, loss.cpu().numpy()[:m], w0, -0.1, 0.1, row_idx=rows)
    assert 0 < z.sum() < m
    tol = 1e-4 * np.abs(w_ref) + 1e-4 * math.sqrt(float(np.mean(w_ref.astype(np.float64) ** 2)))
    assert np.all(np.abs(w.cpu().numpy() - w_ref) <= tol)
    assert abs(b.item() - float(b_ref)) <= 1e-4 * abs(float(b_ref)) + 1e-7


def test_conv_argument_checks(aa):
    x = W.normal((4, 3 * 8 * 8), 1.0, 1, torch.float32, DEV)
    wt = torch.zeros((2, 3, 3, 3), device=DEV)
    phi = torch.zeros((4, 2 * 16), device=DEV)
    with pytest.raises(B.AutoAssistError) as e:
        aa.aa_conv_pool_features(B.dense_features(x), B.conv_layer(wt, None, 8, 8, 3), phi)      # pool does not divide the image
    assert e.value.status == B.AA_ERR_INVALID_ARG
    with pytest.raises(B.AutoAssistError) as e:
        aa.aa_conv_pool_features(B.dense_features(x), B.conv_layer(wt, None, 8, 16, 2), phi)     # image size does not match d
    assert e.value.status == B.AA_ERR_INVALID_ARG
    with pytest.raises(B.AutoAssistError) as e:
        aa.aa_conv_pool_features(B.dense_features(x), B.conv_layer(torch.zeros((2, 3, 7, 7), device=DEV), None, 8, 8, 2), phi)
    assert e.value.status == B.AA_ERR_UNSUPPORTED
