"""The workloads at their full sizes, in the launch configurations that are timed.

The oracle checks sampled outputs (rows it can compute one by one); what cannot be sampled is covered by properties
that hold at any size (list == nonzero(mask), acceptance statistics, additivity of gradients over sub-batches).
Tolerances are those of test_gpu_parity.py / test_gpu_mlp.py.
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


def sample_rows(n, k, seed):
    return np.unique(np.concatenate([np.arange(40), np.arange(n - 40, n),
                                     np.random.default_rng(seed).integers(0, n, k)])).astype(np.int64)


def rows_of(t, sample):
    return t[torch.from_numpy(sample).to(t.device)]


def test_image_shape_loss_and_assistant_step_full_size():
    """Image shape: 100-class losses of a 36,000-row batch and the Assistant step on those rows of a 65,536 x 3072 pool."""
    build.build()
    cfg = W.ImageShape()
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, device=DEV)
    x = cfg.pool(1, DEV)
    m = 36000
    rows = np.sort(np.random.default_rng(1).permutation(cfg.n)[:m]).astype(np.int32)
    rows_t = torch.from_numpy(rows).to(DEV)
    logits, labels = cfg.logits(1, DEV), cfg.labels(1, DEV)
    loss = torch.zeros(cfg.n, dtype=torch.float32, device=DEV)
    cnt = torch.tensor([m], dtype=torch.int32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits), labels, loss, count_dev=cnt)
    torch.cuda.synchronize()
    f_ref = O.row_loss(W.to_oracle(logits[:m]), labels[:m].cpu().numpy())
    f_gpu = loss[:m].cpu().numpy()
    assert np.max(np.abs(f_gpu - f_ref)) <= 1e-4
    w, b = cfg.assistant(DEV)
    w0 = w.cpu().numpy().copy()
    aa.aa_assistant_step(B.dense_features(x, row_idx=rows_t), loss, B.linear_assistant(w, b), cfg.lr, count_dev=cnt)
    torch.cuda.synchronize()
    assert aa.aa_device_status() == B.AA_OK
    w_ref, b_ref, z = O.assistant_step_linear_dense(W.to_oracle(x), f_gpu, w0, 0.0, cfg.lr, row_idx=rows)
    assert 0 < z.sum() < m
    tol = 1e-4 * np.abs(w_ref) + 1e-4 * math.sqrt(float(np.mean(w_ref.astype(np.float64) ** 2)))
    assert np.all(np.abs(w.cpu().numpy() - w_ref) <= tol)
    assert abs(b.item() - float(b_ref)) <= 1e-4 * abs(float(b_ref)) + 1e-7
    aa.close()


def test_translation_shape_full_size():
    """Translation shape: bag-of-words screen of 16,384 sentences, then 25,000 x 32,000 bf16 token logits summed per sentence."""
    build.build()
    cfg = W.TranslationShape()
    aa = B.AutoAssist(max_rows=max(cfg.n, cfg.token_budget), max_d=cfg.buckets, device=DEV)
    indptr, col, val, lengths = cfg.csr(DEV)
    w, b = cfg.assistant(DEV)
    out_idx = torch.full((cfg.n,), -7, dtype=torch.int32, device=DEV)
    out_count = torch.zeros(1, dtype=torch.int32, device=DEV)
    out_score = torch.zeros(cfg.n, dtype=torch.float32, device=DEV)
    out_mask = torch.zeros(cfg.n, dtype=torch.uint8, device=DEV)
    aa.aa_score_shrink(B.csr_features(indptr, col, val, cfg.buckets), B.linear_assistant(w, b), cfg.gamma, cfg.philox_seed, 5,
                       out_idx, out_count, out_score, out_mask)
    torch.cuda.synchronize()
    ip, cc, vv = indptr.cpu().numpy(), col.cpu().numpy(), val.cpu().numpy()
    wh = w.cpu().numpy()
    s_ref = O.score_csr(ip, cc, vv, wh, 0.0)
    scale = np.sqrt(np.diff(ip).astype(np.float64)) * float(np.linalg.norm(wh))
    s = out_score.cpu().numpy()
    assert np.all(np.abs(s - s_ref) <= 1e-5 * (np.abs(s_ref) + scale))
    g = O.sigmoid(s_ref)
    c = O.uniform(cfg.philox_seed, 5, np.arange(cfg.n))
    far = np.abs(O.accept_prob(g, cfg.gamma) - c) >= 1e-5
    mask = out_mask.cpu().numpy()
    assert np.array_equal(mask[far], O.shrink(g, cfg.gamma, cfg.philox_seed, 5)[far])
    m = int(out_count.item())
    assert m == int(mask.sum()) and np.array_equal(out_idx.cpu().numpy()[:m], O.compact(mask))
    assert abs(m / cfg.n - 0.6) < 0.02          # zero-ish weights: gamma + (1 - gamma) / 2
    # the batch: first accepted sentences within the token budget; one logit row per target token
    batch = out_idx.cpu().numpy()[:m]
    off = W.token_budget_offsets(lengths.cpu().numpy()[batch], cfg.token_budget)
    rows = int(off[-1])
    assert 24800 < rows <= cfg.token_budget and len(off) - 1 > 300
    logits = cfg.token_logits(rows, DEV)
    ids = cfg.token_ids(rows, DEV)
    sent = torch.zeros(len(off) - 1, dtype=torch.float32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits), ids, sent, offsets=torch.from_numpy(off).to(DEV))
    torch.cuda.synchronize()
    got = sent.cpu().numpy()
    # oracle on sampled sentences (all their token rows)
    pick = np.unique(np.concatenate([[0, len(off) - 2], np.random.default_rng(2).integers(0, len(off) - 1, 6)]))
    for sidx in pick:
        a, e = int(off[sidx]), int(off[sidx + 1])
        ell = O.row_loss(W.to_oracle(logits[a:e]), ids[a:e].cpu().numpy())
        assert abs(got[sidx] - ell.sum()) <= 1e-4 * max(1, e - a)
    assert np.all(got > 0) and abs(got.sum() / rows - (math.log(cfg.vocab) + 8.0)) < 1.0   # E[loss] ~ ln V + sigma^2 / 2 for N(0, 4) logits
    assert aa.aa_device_status() == B.AA_OK
    aa.close()


@pytest.mark.parametrize("log2n,mix", [(20, 0.05), (22, 0.5), (24, 0.05)])
def test_scaling_sweep_pools(log2n, mix):
    """Scaling sweep: fp32 d = 512 pools of 2^20 .. 2^24 instances, fused screen and screen from stored scores."""
    build.build()
    n, d = 1 << log2n, 512
    aa = B.AutoAssist(max_rows=n, max_d=d, device=DEV)
    x = torch.randn((n, d), device=DEV, dtype=torch.float32, generator=torch.Generator(device=DEV).manual_seed(14 + log2n))
    w, b = W.linear_assistant(d, 2, DEV)
    out_idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    out_count = torch.zeros(1, dtype=torch.int32, device=DEV)
    out_score = torch.zeros(n, dtype=torch.float32, device=DEV)
    out_mask = torch.zeros(n, dtype=torch.uint8, device=DEV)
    base = (1 << 33) + 5
    aa.aa_score_shrink(B.dense_features(x, id_base=base), B.linear_assistant(w, b), mix, 3, 9, out_idx, out_count, out_score, out_mask)
    torch.cuda.synchronize()
    m = int(out_count.item())
    # integer work at any size: the list is nonzero(mask), ascending, complete
    nz = torch.nonzero(out_mask).flatten().to(torch.int32)
    assert m == nz.numel() and torch.equal(out_idx[:m], nz) and bool((out_idx[m:] == -7).all())
    sample = sample_rows(n, 2000, log2n)
    xs = rows_of(x, sample)
    wh = w.cpu().numpy()
    s_ref = O.score_dense(W.to_oracle(xs), wh, 0.0)
    xn = np.linalg.norm(xs.double().cpu().numpy(), axis=1)
    s = out_score.cpu().numpy()
    assert np.all(np.abs(s[sample] - s_ref) <= 1e-5 * (np.abs(s_ref) + np.linalg.norm(wh) * xn))
    g = O.sigmoid(s_ref)
    c = O.uniform(3, 9, sample + base)
    keep = O.shrink(g, mix, 3, 9, id_base=base, row_idx=sample.astype(np.int32)) if n <= (1 << 31) else None
    far = np.abs(O.accept_prob(g, mix) - c) >= 1e-5
    assert np.array_equal(out_mask.cpu().numpy()[sample][far], keep[far])
    p_all = O.accept_prob(O.sigmoid(s.astype(np.float64)), mix)
    assert abs(m - p_all.sum()) < 5 * math.sqrt((p_all * (1 - p_all)).sum())
    # the split variant on the stored scores gives the same batch
    idx2 = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    cnt2 = torch.zeros(1, dtype=torch.int32, device=DEV)
    aa.aa_shrink_compact(out_score, mix, 3, 9, idx2, cnt2, id_base=base)
    torch.cuda.synchronize()
    assert int(cnt2.item()) == m and torch.equal(idx2, out_idx)
    assert aa.aa_device_status() == B.AA_OK
    aa.close()


@pytest.mark.parametrize("rows,vocab,ragged", [(16384, 131072, True), (65536, 8192, False), (4096, 32768, True)])
def test_loss_sweep_shapes(rows, vocab, ragged):
    build.build()
    aa = B.AutoAssist(max_rows=rows, max_d=8, device=DEV)
    logits = W.sweep_logits(rows, vocab, DEV)
    ids = W.randint(0, vocab, (rows,), 16, DEV)
    out = torch.zeros(rows, dtype=torch.float32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits), ids, out)
    torch.cuda.synchronize()
    sample = sample_rows(rows, 40, vocab)
    ell = O.row_loss(W.to_oracle(rows_of(logits, sample)), rows_of(ids, sample).cpu().numpy())
    got = out.cpu().numpy()
    assert np.max(np.abs(got[sample] - ell)) <= 1e-4
    if ragged:
        off = W.ragged_offsets(rows, 8, 128, 17)
        sent = torch.zeros(len(off) - 1, dtype=torch.float32, device=DEV)
        aa.aa_instance_loss(B.logits_desc(logits), ids, sent, offsets=torch.from_numpy(off).to(DEV))
        torch.cuda.synchronize()
        # per-sentence sums against the (verified-by-sample) row losses of the same kernel, added in fp64
        ref = np.add.reduceat(got.astype(np.float64), off[:-1])
        assert np.all(np.abs(sent.cpu().numpy() - ref) <= 1e-4 * np.maximum(1, np.diff(off)))
    assert aa.aa_device_status() == B.AA_OK
    aa.close()


def test_mlp_shape_loss_and_step_full_size():
    """MLP shape: 1000-class losses of a 144,000-row batch (sampled), and the two-layer step on that batch: its update must be
    the row-weighted sum of the updates of eight sub-batches taken from the same parameters (additivity of the mean gradient),
    which ties the full-size launch geometry to sizes the oracle checks directly in test_gpu_mlp.py."""
    build.build()
    cfg = W.MlpShape()
    m = 144000
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, max_hidden=cfg.hidden, device=DEV)
    logits, labels = cfg.logits(m, DEV), cfg.labels(m, DEV)
    loss = torch.zeros(m, dtype=torch.float32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits), labels, loss)
    torch.cuda.synchronize()
    sample = sample_rows(m, 300, 5)
    ell = O.row_loss(W.to_oracle(rows_of(logits, sample)), rows_of(labels, sample).cpu().numpy())
    assert np.max(np.abs(loss.cpu().numpy()[sample] - ell)) <= 1e-4
    del logits
    x = cfg.pool(DEV)
    rows = torch.sort(torch.randperm(cfg.n, device=DEV, generator=torch.Generator(device=DEV).manual_seed(6))[:m]).values.to(torch.int32)
    W1, b1, w2, b2 = cfg.assistant(DEV)
    b1 = W.normal((cfg.hidden,), 0.1, 20, torch.float32, DEV)
    T, lr = 7.5, 0.5

    def step(sel_rows, sel_loss):
        P = [W1.clone(), W1.to(torch.bfloat16).contiguous(), b1.clone(), w2.clone(), b2.clone()]
        aa.aa_assistant_step(B.dense_features(x, row_idx=sel_rows.contiguous()), sel_loss.contiguous(), B.mlp_assistant(*P), lr, threshold=T)
        torch.cuda.synchronize()
        return [(a.double() - b_.double()) for a, b_ in zip((W1, b1, w2, b2), (P[0], P[2], P[3], P[4]))]   # lr * mean gradient

    full = step(rows, loss)
    parts = [torch.zeros_like(t) for t in full]
    k = 8
    for q in range(k):
        a, e = q * m // k, (q + 1) * m // k
        for acc, dlt in zip(parts, step(rows[a:e], loss[a:e])):
            acc += dlt * ((e - a) / m)
    assert aa.aa_device_status() == B.AA_OK
    for name, f_, p_ in zip(("W1", "b1", "w2", "b2"), full, parts):
        scale = float(p_.abs().max())
        assert scale > 0, name
        # both sides round P to bf16 identically (same rows, same parameters); what differs is the fp32 summation order
        assert float((f_ - p_).abs().max()) <= 2e-4 * scale, (name, float((f_ - p_).abs().max()), scale)
    aa.close()


def test_conv_shape_full_size_sampled():
    """Convolutional Assistant at the size that is timed (65,536 images of 3 x 32 x 32 bf16, 16 channels of 3 x 3 taps,
    4 x 4 pooling): the oracle evaluates sampled images; the bar is the one of test_gpu_conv.py."""
    build.build()
    cfg = W.ConvShape()
    x = cfg.pool_images(0, DEV)
    weight, bias = cfg.conv(DEV)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=max(cfg.d, cfg.features), device=DEV)
    phi = torch.full((cfg.n, cfg.features), -9.0, dtype=torch.float32, device=DEV)
    aa.aa_conv_pool_features(B.dense_features(x), B.conv_layer(weight, bias, cfg.height, cfg.width, cfg.pool), phi)
    torch.cuda.synchronize()
    assert aa.aa_device_status() == B.AA_OK
    sample = sample_rows(cfg.n, 120, 9)
    xs = rows_of(x, sample).contiguous()
    ref = O.conv_pool_features(W.to_oracle(xs), cfg.c_in, cfg.height, cfg.width, weight.cpu().numpy(), bias.cpu().numpy(), cfg.pool)
    scale = O.conv_pool_features(W.to_oracle(xs.abs()), cfg.c_in, cfg.height, cfg.width, weight.abs().cpu().numpy(),
                                 bias.abs().cpu().numpy(), cfg.pool)
    got = rows_of(phi, sample).cpu().numpy()
    err = np.abs(got - ref)
    assert np.all(err <= 1e-5 * (np.abs(ref) + scale) + 1e-30), float(np.max(err / (np.abs(ref) + scale + 1e-30)))
    assert float(phi.min()) >= 0.0 and ref.std() > 0.01          # every image was written (rectified values, no -9 left)
    aa.close()


def test_mlp_scored_step_full_size_equals_the_recomputing_step():
    """Two-layer Assistant at the size that is timed (262,144 x 3072 pool, hidden 256): the update that takes the
    screening's scores and gate bits must give the parameters of the update that evaluates the forward pass itself, on
    the batch the screening produced.  Both routes are tied to the oracle at 40,000 rows in test_gpu_mlp.py; here the
    full-size launch geometry of the scored route is tied to the other one."""
    build.build()
    cfg = W.MlpShape()
    x = cfg.pool(DEV)
    W1, b1, w2, b2 = cfg.assistant(DEV)
    b1 = W.normal((cfg.hidden,), 0.1, 21, torch.float32, DEV)
    aa = B.AutoAssist(max_rows=cfg.n, max_d=cfg.d, max_hidden=cfg.hidden, device=DEV)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    score = torch.zeros(cfg.n, dtype=torch.float32, device=DEV)
    loss = (W.normal((cfg.n,), 1.0, 22, torch.float32, DEV).abs() * 2).contiguous()
    feat, batch = B.dense_features(x), B.dense_features(x, row_idx=out_idx)

    def fresh():
        return [W1.clone(), W1.to(torch.bfloat16).contiguous(), b1.clone(), w2.clone(), b2.clone()]

    P = fresh()
    aa.aa_score_shrink(feat, B.mlp_assistant(*P), cfg.gamma, cfg.philox_seed, 2, out_idx, cnt, score)
    aa.aa_assistant_step_scored(batch, loss, score, B.mlp_assistant(*P), 0.5, count_dev=cnt)
    Q = fresh()
    aa.aa_assistant_step(batch, loss, B.mlp_assistant(*Q), 0.5, count_dev=cnt)
    torch.cuda.synchronize()
    assert aa.aa_device_status() == B.AA_OK
    m = int(cnt.item())
    assert 100000 < m < cfg.n
    start = fresh()
    for name, got, want, was in zip(("W1", "W1_bf16", "b1", "w2", "b2"), P, Q, start):
        step = (want.double() - was.double())
        scale = float(step.abs().max())
        assert scale > 0, name
        # the same rows, gates and residuals on both routes; what differs is fp32 summation order (and, for w2, the
        # identity that takes sum_i r_i relu(a_iu) from the W1-gradient contraction)
        tol = 2e-4 * scale if name != "W1_bf16" else 2.0 ** -7 * float(want.double().abs().max())
        assert float((got.double() - want.double()).abs().max()) <= tol, (name, float((got.double() - want.double()).abs().max()), scale)
    aa.close()
