"""Parity of the two-layer (tensor-core) Assistant with the CPU oracle.

Bars: pre-activation scores |s - s_ref| <= 1e-5 (|s_ref| + sum_j |w2_j| ||W1_j|| ||x_i||), i.e. relative to the
scale of the terms the two layers add up (bf16 products are exact in fp32; only the accumulation order differs);
keep/skip mask bit-exact outside the tie band |p - c| < 1e-5; batch list bit-exact given the mask.
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
    ctx = B.AutoAssist(max_rows=1 << 19, max_d=4096, max_hidden=256, device=DEV)
    yield ctx
    torch.cuda.synchronize()
    assert ctx.aa_device_status() == B.AA_OK
    ctx.close()


def bf16_values(t):
    """fp64 NumPy array of the values a bf16 tensor holds."""
    return t.float().double().cpu().numpy()


def make_mlp(d, hidden, seed, b1_std=0.2, b2=0.1):
    W1, b1, w2, _ = W.mlp_assistant(d, hidden, seed, DEV)
    b1 = W.normal((hidden,), b1_std, seed + 5, torch.float32, DEV)
    b2_t = torch.full((1,), b2, dtype=torch.float32, device=DEV)
    W1b = W1.to(torch.bfloat16).contiguous()
    return W1, W1b, b1, w2, b2_t


def mlp_screen(aa, x, params, mix, seed, step, id_base=0):
    W1, W1b, b1, w2, b2 = params
    n = x.shape[0]
    out_idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    out_count = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    out_score = torch.zeros(n, dtype=torch.float32, device=DEV)
    out_mask = torch.full((n,), 9, dtype=torch.uint8, device=DEV)
    aa.aa_score_shrink(B.dense_features(x, id_base=id_base), B.mlp_assistant(W1, W1b, b1, w2, b2), mix, seed, step,
                       out_idx, out_count, out_score, out_mask)
    torch.cuda.synchronize()
    return out_idx.cpu().numpy(), int(out_count.item()), out_score.cpu().numpy(), out_mask.cpu().numpy()


def check_against_oracle(gpu, x_rows, params, mix, seed, step, ids):
    """x_rows: the bf16 rows (tensor) the oracle scores; ids: their instance ids."""
    idx, m, s, mask = gpu
    W1, W1b, b1, w2, b2 = params
    W1v = bf16_values(W1b)
    s_ref = O.score_mlp(W.to_oracle(x_rows.contiguous()), W1v, b1.cpu().numpy(), w2.cpu().numpy(), float(b2.item()))
    xn = np.linalg.norm(bf16_values(x_rows), axis=1)
    scale = float(np.sum(np.abs(w2.double().cpu().numpy()) * np.linalg.norm(W1v, axis=1))) * xn
    tol = 1e-5 * (np.abs(s_ref) + scale)
    assert np.all(np.abs(s - s_ref) <= tol), float(np.max(np.abs(s - s_ref) / tol))
    g = O.sigmoid(s_ref)
    p = O.accept_prob(g, mix)
    c = O.uniform(seed, step, ids)
    keep = O.shrink(g, mix, seed, step, row_idx=np.asarray(ids, np.int32))
    far = np.abs(p - c) >= 1e-5
    return s_ref, keep, far


@pytest.mark.parametrize("n,d,hidden", [
    (1, 64, 16), (255, 64, 64), (257, 192, 32), (1000, 200, 64), (777, 3072, 256), (2048, 1000, 256), (5000, 128, 240),
])
def test_mlp_screen_matches_the_oracle(aa, n, d, hidden):
    x = W.normal((n, d), 1.0, 90 + n, torch.bfloat16, DEV)
    params = make_mlp(d, hidden, 91 + d)
    mix, seed, step = 0.1, 7, n
    gpu = mlp_screen(aa, x, params, mix, seed, step)
    idx, m, s, mask = gpu
    ids = np.arange(n)
    s_ref, keep, far = check_against_oracle(gpu, x, params, mix, seed, step, ids)
    assert set(np.unique(mask)) <= {0, 1}
    assert np.array_equal(mask[far], keep[far])
    assert m == int(mask.sum()) and np.array_equal(idx[:m], O.compact(mask))
    assert np.all(idx[m:] == -7)
    assert np.std(s_ref) > 0.05 or n == 1      # the case exercises a non-trivial score range


def test_mlp_reduces_to_known_forms_on_the_gpu(aa):
    # selector W1 (unit rows), w2 = 1, zero biases: s_i = sum_j relu(x_ij) over the first `hidden` features
    n, d, hidden = 600, 128, 64
    x = W.normal((n, d), 1.0, 5, torch.bfloat16, DEV)
    W1 = torch.zeros((hidden, d), device=DEV)
    W1[torch.arange(hidden), torch.arange(hidden)] = 1.0
    params = (W1, W1.to(torch.bfloat16), torch.zeros(hidden, device=DEV), torch.ones(hidden, device=DEV), torch.zeros(1, device=DEV))
    _, _, s, _ = mlp_screen(aa, x, params, 0.1, 1, 1)
    expect = torch.relu(x[:, :hidden].float()).double().sum(1).cpu().numpy()
    assert np.max(np.abs(s - expect)) <= 1e-5 * (np.abs(expect).max() + 1)


def test_mlp_strided_rows_offset_ids_and_repeatability(aa):
    n, d, hidden = 3000, 256, 128
    buf = W.normal((n, d + 8), 1.0, 6, torch.bfloat16, DEV)
    x = buf[:, :d]                                   # row stride d + 8 elements (16-byte aligned)
    params = make_mlp(d, hidden, 17)
    base = (1 << 32) - 77
    gpu = mlp_screen(aa, x, params, 0.3, (1 << 40) + 1, 12, id_base=base)
    idx, m, s, mask = gpu
    W1, W1b, b1, w2, b2 = params
    s_ref = O.score_mlp(W.to_oracle(x.contiguous()), bf16_values(W1b), b1.cpu().numpy(), w2.cpu().numpy(), float(b2.item()))
    g = O.sigmoid(s_ref)
    keep = O.shrink(g, 0.3, (1 << 40) + 1, 12, id_base=base)
    c = O.uniform((1 << 40) + 1, 12, np.arange(n) + base)
    far = np.abs(O.accept_prob(g, 0.3) - c) >= 1e-5
    assert np.array_equal(mask[far], keep[far])
    assert m == int(mask.sum()) and np.array_equal(idx[:m], O.compact(mask))
    again = mlp_screen(aa, x, params, 0.3, (1 << 40) + 1, 12, id_base=base)
    assert again[1] == m and np.array_equal(again[0], idx) and np.array_equal(again[2], s)


def test_mlp_candidate_list_gathers_rows(aa):
    n_store, n, d, hidden = 1500, 1000, 320, 96
    x = W.normal((n_store, d), 1.0, 30, torch.bfloat16, DEV)
    params = make_mlp(d, hidden, 31)
    W1, W1b, b1, w2, b2 = params
    rows = np.random.default_rng(32).permutation(n_store)[:n].astype(np.int32)
    rows_t = torch.from_numpy(rows).to(DEV)
    out_idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    out_count = torch.zeros(1, dtype=torch.int32, device=DEV)
    out_score = torch.zeros(n, dtype=torch.float32, device=DEV)
    out_mask = torch.zeros(n, dtype=torch.uint8, device=DEV)
    aa.aa_score_shrink(B.dense_features(x, row_idx=rows_t, id_base=10), B.mlp_assistant(W1, W1b, b1, w2, b2), 0.2, 3, 4,
                       out_idx, out_count, out_score, out_mask)
    torch.cuda.synchronize()
    m, s, mask, idx = int(out_count.item()), out_score.cpu().numpy(), out_mask.cpu().numpy(), out_idx.cpu().numpy()
    W1v = bf16_values(W1b)
    s_ref = O.score_mlp(W.to_oracle(x), W1v, b1.cpu().numpy(), w2.cpu().numpy(), float(b2.item()), row_idx=rows)
    xn = np.linalg.norm(bf16_values(x)[rows], axis=1)
    scale = float(np.sum(np.abs(w2.double().cpu().numpy()) * np.linalg.norm(W1v, axis=1))) * xn
    assert np.all(np.abs(s - s_ref) <= 1e-5 * (np.abs(s_ref) + scale))
    g = O.sigmoid(s_ref)
    keep = O.shrink(g, 0.2, 3, 4, id_base=10, row_idx=rows)
    c = O.uniform(3, 4, rows.astype(np.int64) + 10)
    far = np.abs(O.accept_prob(g, 0.2) - c) >= 1e-5
    assert np.array_equal(mask[far], keep[far])
    assert m == int(mask.sum()) and np.array_equal(idx[:m], O.compact(mask, row_idx=rows))
    # an entry outside the stored rows is skipped and latched
    bad = rows_t.clone(); bad[5] = n_store; bad[700] = -3
    aa.aa_score_shrink(B.dense_features(x, row_idx=bad, id_base=10), B.mlp_assistant(W1, W1b, b1, w2, b2), 1.0, 3, 4,
                       out_idx, out_count, out_score, out_mask)
    torch.cuda.synchronize()
    mask = out_mask.cpu().numpy()
    assert mask[5] == 0 and mask[700] == 0 and int(out_count.item()) == n - 2
    assert aa.aa_device_status() == B.AA_ERR_BAD_INDEX


def params_close(got, ref, what, slack=None):
    ref = np.asarray(ref, np.float64).reshape(-1)
    got = np.asarray(got, np.float64).reshape(-1)
    tol = 1e-4 * np.abs(ref) + 1e-4 * math.sqrt(float(np.mean(ref ** 2)) + 1e-300)
    if slack is not None:
        tol = tol + slack
    err = np.abs(got - ref)
    assert np.all(err <= tol), (what, float(np.max(err - tol)))


@pytest.mark.parametrize("n,m,d,hidden,use_rows,thr,lr", [
    (300, 300, 64, 16, False, None, 0.1), (2000, 1500, 192, 64, True, None, 0.1), (1000, 1000, 200, 256, False, 1.5, 0.1),
    (5000, 2777, 3072, 256, True, None, 0.05), (700, 1, 128, 32, True, None, 0.1), (1300, 1300, 600, 128, False, None, 1.0),
])
def test_mlp_assistant_step(aa, n, m, d, hidden, use_rows, thr, lr):
    check_mlp_step(aa, n, m, d, hidden, use_rows, thr, lr)


def test_mlp_assistant_step_many_tiles_per_cta_and_every_split(aa):
    """40,000 batch rows picked out of a 65,536 x 3072 pool, hidden 256: every CTA of the forward pass runs several
    128-row tiles through both of its alternating accumulators, and every split-K slice of the W1-gradient kernel
    carries some fifty 64-row slices.  The whole step is checked against the oracle (about a minute of CPU time)."""
    check_mlp_step(aa, 65536, 40000, 3072, 256, True, None, 0.01)


def check_mlp_step(aa, n, m, d, hidden, use_rows, thr, lr, scored=None):
    """scored: None = the step evaluates the forward pass itself; "screen" = the pool is screened first on the same context
    and the step gets that screening's scores; "altered" = as "screen", but the scores are changed on the way (the oracle
    gets the same changed scores: the step must really be using what it is handed)."""
    rng = np.random.default_rng(n + d)
    x = W.normal((n, d), 1.0, 60 + d, torch.bfloat16, DEV)
    W1, W1b, b1, w2, b2 = make_mlp(d, hidden, 61 + d)
    loss = (W.normal((m,), 1.0, 62, torch.float32, DEV).abs() * 2).contiguous()
    rows = np.sort(rng.permutation(n)[:m]).astype(np.int32) if use_rows else None
    rows_t = None if rows is None else torch.from_numpy(rows).to(DEV)
    host = {k: v.cpu().numpy().copy() for k, v in (("W1", W1), ("b1", b1), ("w2", w2))}
    b2_0 = float(b2.item())
    W1b_bits = W.to_oracle(W1b).copy()
    W1b_before = W1b.clone()
    feat = B.dense_features(x, row_idx=rows_t) if use_rows else B.dense_features(x[:m])
    cnt = torch.tensor([m], dtype=torch.int32, device=DEV)
    s_given = None
    if scored is None:
        aa.aa_assistant_step(feat, loss, B.mlp_assistant(W1, W1b, b1, w2, b2), lr, threshold=thr, count_dev=cnt)
    else:
        assert use_rows or m == n                        # the scores are those of the pool's stored rows
        sink_idx = torch.zeros(n, dtype=torch.int32, device=DEV)
        sink_cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
        score = torch.zeros(n, dtype=torch.float32, device=DEV)
        asst = B.mlp_assistant(W1, W1b, b1, w2, b2)
        aa.aa_score_shrink(B.dense_features(x), asst, 0.3, 5, 1, sink_idx, sink_cnt, score)
        if scored == "altered":
            score = (score * 0.5 + 0.3).contiguous()
            s_given = score.cpu().numpy().astype(np.float64)
            s_given = s_given[rows] if use_rows else s_given
        aa.aa_assistant_step_scored(feat, loss, score, asst, lr, threshold=thr, count_dev=cnt)
    torch.cuda.synchronize()
    assert aa.aa_device_status() == B.AA_OK
    ref = O.assistant_step_mlp(W.to_oracle(x), loss.cpu().numpy(), host["W1"], W1b_bits, host["b1"], host["w2"], b2_0, lr,
                               T=thr, row_idx=rows, s=s_given)
    # The gate [a > 0] is a decision that floating point takes: fp32 accumulation on the GPU, fp64 in the oracle.  Where the
    # oracle's pre-activation lies within the score tolerance of zero (1e-5 of the scale of its terms) either decision is
    # valid, and the W1 gradient may differ by that row's whole contribution; everywhere else the updated W1 is held to the
    # plain bar.  r enters the contraction as two bf16 terms (relative error 2^-17 of each row's contribution).
    gW1 = ref["grads"][0]
    xs = bf16_values(x[:m] if rows is None else x[rows_t.long()])
    r = O.sigmoid(ref["s"] if s_given is None else s_given) - ref["z"]
    on = ref["a"] > 0
    W1v = bf16_values(W1b_before)
    a_scale = np.abs(host["b1"].astype(np.float64))[None, :] + np.linalg.norm(xs, axis=1)[:, None] * np.linalg.norm(W1v, axis=1)[None, :]
    near = np.abs(ref["a"]) <= 1e-5 * a_scale
    w2h = host["w2"].astype(np.float64)
    kink = (np.abs(r)[:, None] * near).T @ np.abs(xs) * np.abs(w2h)[:, None] / m
    bound = (np.abs(r)[:, None] * on).T @ np.abs(xs) * np.abs(w2h)[:, None] / m * 2.0 ** -16 + kink
    assert near.mean() < 1e-3                       # such ties are rare: the slack below is zero for all but a few weights
    # parameters after the update: rel 1e-4 (+ 1e-4 rms floor), for every batch size and step size
    params_close(W1.cpu().numpy(), ref["W1"], "W1", slack=lr * kink.reshape(-1) if near.any() else None)
    params_close(b1.cpu().numpy(), ref["b1"], "b1")
    params_close(w2.cpu().numpy(), ref["w2"], "w2")
    params_close([b2.item()], [ref["b2"]], "b2")
    # the bf16 copy is the nearest-even rounding of the GPU's own new master
    assert np.array_equal(W.to_oracle(W1b), O.round_bf16(W1.cpu().numpy()))
    assert np.abs(W1.cpu().numpy() - host["W1"]).max() > 0
    # the gradient itself, recovered from the update (which is rounded once to fp32)
    g_gpu = (host["W1"].astype(np.float64) - W1.double().cpu().numpy()) / lr
    ulp = np.abs(host["W1"]) * 2.0 ** -23 / lr
    fp32 = 1e-6 * (np.abs(r)[:, None] * on).T @ np.abs(xs) * np.abs(w2h)[:, None] / m     # fp32 accumulation over the batch rows
    assert np.all(np.abs(g_gpu - gW1) <= bound + fp32 + 2 * ulp + 1e-12), float(np.max(np.abs(g_gpu - gW1) - bound - fp32 - 2 * ulp))


@pytest.mark.parametrize("scored", ["screen", "altered"])
@pytest.mark.parametrize("n,m,d,hidden,use_rows,thr,lr", [
    (2000, 1500, 256, 64, True, None, 0.1), (1000, 1000, 384, 256, False, 1.5, 0.1), (5000, 2777, 3072, 256, True, None, 0.05),
    (700, 1, 128, 32, True, None, 0.1), (1300, 1300, 640, 128, False, None, 1.0), (900, 333, 128, 16, True, None, 0.1),
])
def test_mlp_assistant_step_on_the_scores_and_gates_of_the_screening(aa, n, m, d, hidden, use_rows, thr, lr, scored):
    """The update right after a screening on the same context: r from the screening's scores, the gates [a > 0] from
    the bits it left in the workspace, grad w2 through  sum_k W1b_uk G_uk + b1_u sum_i r_i [a_iu > 0].  Same bars as the
    step that evaluates the forward pass itself."""
    check_mlp_step(aa, n, m, d, hidden, use_rows, thr, lr, scored=scored)


def test_mlp_scored_step_many_rows(aa):
    check_mlp_step(aa, 65536, 40000, 3072, 256, True, None, 0.01, scored="screen")


def test_mlp_scored_step_falls_back_when_the_gates_are_not_those_of_the_pool(aa):
    """Scores are only trusted together with the gates of the same screening.  After an update (the gates are stale), for
    other weights or another pool the step evaluates the forward pass itself, bit for bit like aa_assistant_step, and
    never reads the scores."""
    n, d, hidden, lr = 3000, 256, 64, 0.1
    x = W.normal((n, d), 1.0, 71, torch.bfloat16, DEV)
    loss = (W.normal((n,), 1.0, 72, torch.float32, DEV).abs() * 2).contiguous()
    rows_t = torch.arange(0, n, 2, dtype=torch.int32, device=DEV)
    cnt = torch.tensor([rows_t.numel()], dtype=torch.int32, device=DEV)
    garbage = torch.full((n,), float("nan"), dtype=torch.float32, device=DEV)
    sink_idx = torch.zeros(n, dtype=torch.int32, device=DEV)
    sink_cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    score = torch.zeros(n, dtype=torch.float32, device=DEV)
    feat = B.dense_features(x, row_idx=rows_t)

    def fresh():
        return [t.clone() for t in make_mlp(d, hidden, 73)]

    def plain_steps(k):
        p = fresh()
        for _ in range(k):
            aa.aa_assistant_step(feat, loss, B.mlp_assistant(*p), lr, count_dev=cnt)
        torch.cuda.synchronize()
        return p

    # (a) a second scored step without a screening in between: the first one has changed the parameters
    p = fresh()
    aa.aa_score_shrink(B.dense_features(x), B.mlp_assistant(*p), 0.3, 5, 1, sink_idx, sink_cnt, score)
    aa.aa_assistant_step_scored(feat, loss, score, B.mlp_assistant(*p), lr, count_dev=cnt)
    torch.cuda.synchronize()
    after_one = [t.clone() for t in p]
    aa.aa_assistant_step_scored(feat, loss, garbage, B.mlp_assistant(*p), lr, count_dev=cnt)
    torch.cuda.synchronize()
    q = [t.clone() for t in after_one]
    aa.aa_assistant_step(feat, loss, B.mlp_assistant(*q), lr, count_dev=cnt)
    torch.cuda.synchronize()
    for got, want in zip(p, q):
        assert torch.equal(got, want)
    # (b) weights other than the ones the pool was screened with
    p, other = fresh(), fresh()
    aa.aa_score_shrink(B.dense_features(x), B.mlp_assistant(*p), 0.3, 5, 1, sink_idx, sink_cnt, score)
    aa.aa_assistant_step_scored(feat, loss, garbage, B.mlp_assistant(*other), lr, count_dev=cnt)
    torch.cuda.synchronize()
    for got, want in zip(other, plain_steps(1)):
        assert torch.equal(got, want)
    # (c) a screening with a candidate list leaves no usable gates
    p = fresh()
    aa.aa_score_shrink(B.dense_features(x, row_idx=rows_t), B.mlp_assistant(*p), 0.3, 5, 1, sink_idx, sink_cnt, score)
    aa.aa_assistant_step_scored(feat, loss, garbage, B.mlp_assistant(*p), lr, count_dev=cnt)
    torch.cuda.synchronize()
    for got, want in zip(p, plain_steps(1)):
        assert torch.equal(got, want)
    assert aa.aa_device_status() == B.AA_OK


def test_mlp_step_empty_batch_and_zero_lr(aa):
    x = W.normal((400, 64), 1.0, 1, torch.bfloat16, DEV)
    W1, W1b, b1, w2, b2 = make_mlp(64, 32, 2)
    before = [t.clone() for t in (W1, W1b, b1, w2, b2)]
    loss = torch.ones(400, device=DEV)
    zero = torch.zeros(1, dtype=torch.int32, device=DEV)
    asst = B.mlp_assistant(W1, W1b, b1, w2, b2)
    aa.aa_assistant_step(B.dense_features(x), loss, asst, 0.5, count_dev=zero)
    aa.aa_assistant_step(B.dense_features(x), loss, asst, 0.0)
    torch.cuda.synchronize()
    for t, t0 in zip((W1, W1b, b1, w2, b2), before):
        assert torch.equal(t, t0)


def test_mlp_full_size_pool_sampled(aa):
    """The MLP shape at full size (262,144 x 3072, hidden 256) in the launch configuration that is timed."""
    cfg = W.MlpShape()
    x = cfg.pool(DEV)
    W1, b1, w2, b2 = cfg.assistant(DEV)
    params = (W1, W1.to(torch.bfloat16).contiguous(), b1, w2, b2)
    idx, m, s, mask = mlp_screen(aa, x, params, cfg.gamma, cfg.philox_seed, 3)
    assert m == int(mask.sum()) and np.array_equal(idx[:m], np.nonzero(mask)[0])
    sample = np.unique(np.concatenate([np.arange(40), np.arange(cfg.n - 40, cfg.n),
                                       np.random.default_rng(4).integers(0, cfg.n, 300)])).astype(np.int64)
    xs = x[torch.from_numpy(sample).to(DEV)]
    W1v = bf16_values(params[1])
    s_ref = O.score_mlp(W.to_oracle(xs.contiguous()), W1v, b1.cpu().numpy(), w2.cpu().numpy(), 0.0)
    xn = np.linalg.norm(bf16_values(xs), axis=1)
    scale = float(np.sum(np.abs(w2.double().cpu().numpy()) * np.linalg.norm(W1v, axis=1))) * xn
    assert np.all(np.abs(s[sample] - s_ref) <= 1e-5 * (np.abs(s_ref) + scale))
    g = O.sigmoid(s_ref)
    c = O.uniform(cfg.philox_seed, 3, sample)
    keep = O.shrink(g, cfg.gamma, cfg.philox_seed, 3, row_idx=sample.astype(np.int32))
    far = np.abs(O.accept_prob(g, cfg.gamma) - c) >= 1e-5
    assert np.array_equal(mask[sample][far], keep[far])
    p_all = O.accept_prob(O.sigmoid(s.astype(np.float64)), cfg.gamma)
    assert abs(m - p_all.sum()) < 5 * math.sqrt((p_all * (1 - p_all)).sum())
