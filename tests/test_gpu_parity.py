"""Parity of the CUDA library (through its C ABI) with the CPU oracle on the same seeded inputs.

Bars (written out in each test):
  * batch indices and count: bit-exact given the same mask;
  * keep/skip mask: bit-exact except candidates with |p - c| < 1e-5 (fp32 vs fp64 probability);
  * pre-activations: |s - s_ref| <= 1e-5 (|s_ref| + ||w|| ||x_i||);
  * per-row losses: abs 1e-4; per-sentence sums: abs 1e-4 * max(1, tokens in the sentence);
  * Assistant parameters after an update: |w - w_ref| <= 1e-4 |w_ref| + 1e-4 rms(w_ref).
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
    ctx = B.AutoAssist(max_rows=1 << 17, max_d=1 << 18, device=DEV)
    yield ctx
    torch.cuda.synchronize()
    assert ctx.aa_device_status() == B.AA_OK
    ctx.close()


def screen(aa, feat, assistant, n_cand, mix, seed, step, capacity=None):
    cap = n_cand if capacity is None else capacity
    out_idx = torch.full((max(cap, 1),), -7, dtype=torch.int32, device=DEV)
    out_count = torch.full((1,), -7, dtype=torch.int32, device=DEV)
    out_score = torch.zeros(max(n_cand, 1), dtype=torch.float32, device=DEV)
    out_mask = torch.full((max(n_cand, 1),), 9, dtype=torch.uint8, device=DEV)
    aa.aa_score_shrink(feat, assistant, mix, seed, step, out_idx[:cap] if cap else out_idx[:0], out_count,
                       out_score, out_mask)
    torch.cuda.synchronize()
    m = int(out_count.item())
    return out_idx.cpu().numpy(), m, out_score.cpu().numpy()[:n_cand], out_mask.cpu().numpy()[:n_cand]


def check_screen(gpu, ref_s, ref_keep, ref_p, c, rows, w_norm, x_norms):
    """gpu = (idx, m, score, mask); rows = stored row of each candidate."""
    idx, m, s, mask = gpu
    n = len(ref_s)
    # pre-activations
    tol = 1e-5 * (np.abs(ref_s) + w_norm * x_norms)
    assert np.all(np.abs(s - ref_s) <= tol + 1e-30), float(np.max(np.abs(s - ref_s) - tol))
    # decisions: identical outside the tie band
    assert set(np.unique(mask)) <= {0, 1}
    far = np.abs(ref_p - c) >= 1e-5
    assert np.array_equal(mask[far], ref_keep[far])
    # compaction: bit-exact given the mask
    assert m == int(mask.sum())
    assert np.array_equal(idx[:m], O.compact(mask, row_idx=None if rows is None else rows))
    if rows is None and m:
        assert np.all(np.diff(idx[:m]) > 0) and idx[0] >= 0 and idx[m - 1] < n
    assert np.all(idx[m:] == -7)   # nothing written past the count


def dense_case(aa, n, d, dtype, mix, seed, step, *, stride_pad=0, use_rows=False, id_base=0, w_std=0.3, bias=0.1, offset_elems=0):
    rng = np.random.default_rng(1000 + n + d)
    n_store = n + 5 if use_rows else n
    buf = W.normal((n_store, d + stride_pad), 1.0, 17 + n + d, dtype, DEV)
    if offset_elems:
        flat = torch.zeros(buf.numel() + offset_elems, dtype=dtype, device=DEV)
        flat[offset_elems:] = buf.reshape(-1)
        buf = flat[offset_elems:].view(n_store, d + stride_pad)
    x = buf[:, :d]
    w = W.normal((d,), w_std, 3 + d, torch.float32, DEV)
    b = torch.full((1,), bias, dtype=torch.float32, device=DEV)
    rows = None
    if use_rows:
        rows = rng.permutation(n_store)[:n].astype(np.int32)
    rows_t = None if rows is None else torch.from_numpy(rows).to(DEV)
    feat = B.dense_features(x, row_idx=rows_t, id_base=id_base)
    gpu = screen(aa, feat, B.linear_assistant(w, b), n, mix, seed, step)
    xh = W.to_oracle(x.contiguous())
    ref = O.screen_linear_dense(xh, w.cpu().numpy(), bias, mix, seed, step, id_base=id_base, row_idx=rows)
    ids = (np.arange(n) if rows is None else rows.astype(np.int64)) + id_base
    c = O.uniform(seed, step, ids)
    xd = x.double().cpu().numpy()
    xn = np.linalg.norm(xd if rows is None else xd[rows], axis=1)
    check_screen(gpu, ref["s"], ref["keep"], ref["p"], c, rows, float(np.linalg.norm(w.double().cpu().numpy())), xn)
    assert np.array_equal(gpu[0][:gpu[1]], O.compact(gpu[3], row_idx=rows))
    return gpu, ref


# --------------------------------------------------------------------------
# score -> shrink -> compact
# --------------------------------------------------------------------------

def test_tiny_reference_config_screen(aa):
    cfg = W.TinyRef()
    t = cfg.make(DEV)
    feat = B.dense_features(t["x"])
    gpu = screen(aa, feat, B.linear_assistant(t["w"], t["b"]), cfg.n, cfg.gamma, cfg.philox_seed, cfg.step)
    ref = O.screen_linear_dense(W.to_oracle(t["x"]), t["w"].cpu().numpy(), 0.0, cfg.gamma, cfg.philox_seed, cfg.step)
    c = O.uniform(cfg.philox_seed, cfg.step, np.arange(cfg.n))
    xn = np.linalg.norm(t["x"].double().cpu().numpy(), axis=1)
    check_screen(gpu, ref["s"], ref["keep"], ref["p"], c, None, float(t["w"].double().norm()), xn)
    # the plain relative bound (1e-5 of the score itself) wherever the dot product has not cancelled away:
    # |s| at least 5 % of ||w|| ||x|| leaves fp32 accumulation of 64 terms far inside it
    plain = np.abs(ref["s"]) >= 0.05 * float(t["w"].double().norm()) * xn
    assert plain.sum() > cfg.n // 2
    assert np.all(np.abs(gpu[2] - ref["s"])[plain] <= 1e-5 * np.abs(ref["s"])[plain])
    # zero-ish weights: acceptance near gamma + (1 - gamma)/2
    p_mean = ref["p"].mean()
    assert abs(gpu[1] - ref["p"].sum()) < 5 * math.sqrt((ref["p"] * (1 - ref["p"])).sum())
    assert abs(p_mean - 0.55) < 0.01


@pytest.mark.parametrize("n,d,dtype", [
    (1, 1, torch.float32), (31, 3, torch.float32), (33, 64, torch.float32), (1000, 100, torch.float32),
    (4097, 512, torch.float32), (257, 7, torch.bfloat16), (2049, 3072, torch.bfloat16), (640, 264, torch.bfloat16),
    (96, 8200, torch.float32),
])
def test_dense_shapes_and_ragged_tails(aa, n, d, dtype):
    dense_case(aa, n, d, dtype, mix=0.1, seed=5, step=n)


def test_dense_strided_unaligned_gathered_and_offset_ids(aa):
    dense_case(aa, 777, 256, torch.float32, 0.2, 9, 1, stride_pad=4)                 # aligned stride > d
    dense_case(aa, 777, 256, torch.float32, 0.2, 9, 2, stride_pad=3)                 # stride breaks 16-byte alignment
    dense_case(aa, 500, 128, torch.bfloat16, 0.2, 9, 3, offset_elems=1)              # base pointer off by one element
    dense_case(aa, 1500, 96, torch.bfloat16, 0.3, 9, 4, use_rows=True)               # shuffled candidate list
    dense_case(aa, 900, 64, torch.float32, 0.05, (1 << 40) + 3, (1 << 33) + 1, id_base=(1 << 32) - 100)  # 64-bit ids/seed/step


def test_gamma_extremes_and_saturated_assistant(aa):
    g_all, _ = dense_case(aa, 3000, 32, torch.float32, 1.0, 1, 0)
    assert g_all[1] == 3000 and np.array_equal(g_all[0][:3000], np.arange(3000))
    dense_case(aa, 3000, 32, torch.float32, 0.0, 1, 0)
    g_pos, _ = dense_case(aa, 2000, 16, torch.float32, 0.0, 1, 0, w_std=0.0, bias=60.0)    # g = 1: keep all
    assert g_pos[1] == 2000
    g_neg, _ = dense_case(aa, 2000, 16, torch.float32, 0.0, 1, 0, w_std=0.0, bias=-120.0)  # g = 0: keep none
    assert g_neg[1] == 0


def test_empty_pool_and_capacity_overflow(aa):
    x = torch.zeros((0, 8), dtype=torch.float32, device=DEV)
    w, b = torch.zeros(8, device=DEV), torch.zeros(1, device=DEV)
    idx, m, _, _ = screen(aa, B.dense_features(x), B.linear_assistant(w, b), 0, 0.1, 0, 0)
    assert m == 0
    # capacity smaller than the survivors: count exact, prefix written, condition latched
    x = W.normal((5000, 16), 1.0, 1, torch.float32, DEV)
    full = screen(aa, B.dense_features(x), B.linear_assistant(w[:16].repeat(2)[:16].contiguous(), b), 5000, 0.5, 3, 3)
    cut = screen(aa, B.dense_features(x), B.linear_assistant(w[:16].repeat(2)[:16].contiguous(), b), 5000, 0.5, 3, 3, capacity=100)
    assert cut[1] == full[1] > 100
    assert np.array_equal(cut[0][:100], full[0][:100])
    assert aa.aa_device_status() == B.AA_ERR_CAPACITY
    assert aa.aa_device_status() == B.AA_OK   # reading clears it


def test_out_of_range_candidate_row_is_rejected_and_latched(aa):
    x = W.normal((100, 8), 1.0, 1, torch.float32, DEV)
    rows = torch.tensor([0, 5, 100, 7, -1, 99], dtype=torch.int32, device=DEV)
    w, b = torch.zeros(8, device=DEV), torch.full((1,), 50.0, device=DEV)
    idx, m, _, mask = screen(aa, B.dense_features(x, row_idx=rows), B.linear_assistant(w, b), 6, 0.0, 0, 0)
    assert list(mask) == [1, 1, 0, 1, 0, 1] and list(idx[:m]) == [0, 5, 7, 99]
    assert aa.aa_device_status() == B.AA_ERR_BAD_INDEX


def test_scan_is_deterministic_and_reusable_across_calls(aa):
    x = W.normal((50000, 64), 1.0, 2, torch.float32, DEV)
    w, b = W.linear_assistant(64, 2, DEV)
    feat, asst = B.dense_features(x), B.linear_assistant(w, b)
    first = screen(aa, feat, asst, 50000, 0.1, 11, 5)
    for _ in range(5):
        again = screen(aa, feat, asst, 50000, 0.1, 11, 5)
        assert again[1] == first[1] and np.array_equal(again[0], first[0]) and np.array_equal(again[3], first[3])
    other = screen(aa, feat, asst, 50000, 0.1, 11, 6)
    assert not np.array_equal(other[3], first[3])


def test_shrink_compact_from_scores(aa):
    for n, mix in ((1, 0.1), (1023, 0.05), (1025, 0.5), (70001, 0.05)):
        s = W.normal((n,), 2.0, 40 + n, torch.float32, DEV)
        out_idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
        out_count = torch.zeros(1, dtype=torch.int32, device=DEV)
        out_mask = torch.zeros(n, dtype=torch.uint8, device=DEV)
        aa.aa_shrink_compact(s, mix, 77, 3, out_idx, out_count, out_mask, id_base=12345)
        torch.cuda.synchronize()
        m, mask, idx = int(out_count.item()), out_mask.cpu().numpy(), out_idx.cpu().numpy()
        g = O.sigmoid(s.double().cpu().numpy())
        keep = O.shrink(g, mix, 77, 3, id_base=12345)
        p = O.accept_prob(g, mix)
        c = O.uniform(77, 3, np.arange(n) + 12345)
        far = np.abs(p - c) >= 1e-5
        assert np.array_equal(mask[far], keep[far])
        assert m == int(mask.sum()) and np.array_equal(idx[:m], O.compact(mask))


def make_csr(n, d, max_len, seed, empty_every=0):
    rng = np.random.default_rng(seed)
    lens = rng.integers(0 if empty_every else 1, max_len + 1, n)
    if empty_every:
        lens[::empty_every] = 0
    indptr = np.zeros(n + 1, np.int32)
    indptr[1:] = np.cumsum(lens)
    col = rng.integers(0, d, int(indptr[-1])).astype(np.int32)
    val = rng.integers(1, 4, int(indptr[-1])).astype(np.float32)
    return indptr, col, val


# the last three cases are large pools (many tiles per CTA): few buckets, a bucket count that is not a power of two, and the
# translation shape's 2^18 buckets
@pytest.mark.parametrize("n,d,max_len", [(1, 10, 3), (1000, 50, 6), (4099, 1 << 18, 128), (333, 1000, 700),
                                         (20000, 1000, 60), (70001, 5000, 40), (131072, 1 << 18, 300)])
def test_csr_screen(aa, n, d, max_len):
    indptr, col, val = make_csr(n, d, max_len, 50 + n, empty_every=7)
    w = W.normal((d,), 0.2, 51, torch.float32, DEV)
    b = torch.full((1,), -0.2, device=DEV)
    ti, tc, tv = (torch.from_numpy(a).to(DEV) for a in (indptr, col, val))
    if tc.numel() == 0:
        tc, tv = torch.zeros(1, dtype=torch.int32, device=DEV), torch.zeros(1, device=DEV)
    feat = B.csr_features(ti, tc, tv, d, nnz=int(indptr[-1]))
    gpu = screen(aa, feat, B.linear_assistant(w, b), n, 0.2, 4, 8)
    wh = w.cpu().numpy()
    s = O.score_csr(indptr, col, val, wh, -0.2)
    g = O.sigmoid(s)
    c = O.uniform(4, 8, np.arange(n))
    scale = np.array([np.sqrt((val[a:b_] ** 2).sum()) for a, b_ in zip(indptr[:-1], indptr[1:])])
    check_screen(gpu, s, O.shrink(g, 0.2, 4, 8), O.accept_prob(g, 0.2), c, None, float(np.linalg.norm(wh)), scale)


def test_hard_threshold_shrinking(aa):
    """aa_threshold_compact against the oracle: comparisons of fp32 values, bit-exact."""
    for n, T in ((1, 0.5), (1023, 0.0), (70001, 1.0), (70001, 50.0), (120000, float(B.aa_sk_threshold(6.0, 4)))):
        v = (W.normal((n,), 1.0, 80 + n, torch.float32, DEV).abs() * 1.5).contiguous()
        if n > 10:
            v[3] = float("nan"); v[4] = T; v[5] = float("inf")
        idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
        cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
        mask = torch.full((n,), 9, dtype=torch.uint8, device=DEV)
        aa.aa_threshold_compact(v, T, idx, cnt, mask)
        torch.cuda.synchronize()
        keep = O.hard_shrink(v.cpu().numpy(), T)
        m = int(cnt.item())
        assert np.array_equal(mask.cpu().numpy(), keep)
        assert m == int(keep.sum()) and np.array_equal(idx.cpu().numpy()[:m], O.compact(keep)) and bool((idx[m:] == -7).all())
    assert B.aa_sk_threshold(6.0, 4) == O.sk_threshold(6.0, 4) == 1.5
    assert aa.aa_device_status() == B.AA_OK


def test_batch_cut_and_cursor(aa):
    """aa_batch_cut against the oracle's literal walk: integer work, bit-exact."""
    n = 70001
    s = W.normal((n,), 1.5, 77, torch.float32, DEV)
    idx = torch.full((n,), -7, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    aa.aa_shrink_compact(s, 0.2, 5, 6, idx, cnt)
    torch.cuda.synchronize()
    m = int(cnt.item())
    Bfull = idx.cpu().numpy()[:m]
    lengths = W.randint(8, 129, (n,), 78, DEV)
    lengths[int(Bfull[3])] = -4                                   # a negative count is a zero-length sentence
    lh = lengths.cpu().numpy()
    out_m = torch.zeros(1, dtype=torch.int32, device=DEV)
    out_c = torch.zeros(1, dtype=torch.int32, device=DEV)
    off = torch.full((m + 1,), -7, dtype=torch.int32, device=DEV)
    cases = [dict(batch_size=1), dict(batch_size=1000), dict(batch_size=m), dict(batch_size=m + 5), dict(),
             dict(lengths=lengths, token_budget=25000), dict(lengths=lengths, token_budget=25000, batch_size=100),
             dict(lengths=lengths, token_budget=3), dict(lengths=lengths, token_budget=10 ** 8),
             dict(lengths=lengths, token_budget=2 * 10 ** 6)]     # several scan chunks with a carry
    for kw in cases:
        off.fill_(-7)
        use_off = "lengths" in kw
        aa.aa_batch_cut(idx, cnt, n, out_m, out_c, out_offsets=off if use_off else None, **kw)
        torch.cuda.synchronize()
        b_ref, c_ref, off_ref = O.batch_cut(Bfull, n, batch_size=kw.get("batch_size", 0), lengths=lh if use_off else None,
                                            token_budget=kw.get("token_budget", 0))
        assert (int(out_m.item()), int(out_c.item())) == (b_ref, c_ref), kw
        if use_off:
            got = off.cpu().numpy()
            assert np.array_equal(got[:b_ref + 1], off_ref) and np.all(got[b_ref + 1:] == -7)
    # an empty survivor list consumes the whole pool
    zero = torch.zeros(1, dtype=torch.int32, device=DEV)
    aa.aa_batch_cut(idx, zero, n, out_m, out_c, batch_size=10)
    torch.cuda.synchronize()
    assert (int(out_m.item()), int(out_c.item())) == (0, n)
    assert aa.aa_device_status() == B.AA_OK


# --------------------------------------------------------------------------
# per-instance loss
# --------------------------------------------------------------------------

def run_loss(aa, logits, labels, offsets=None, count=None):
    rows = logits.shape[0]
    n_out = rows if offsets is None else len(offsets) - 1
    out = torch.full((max(n_out, 1),), -3.0, dtype=torch.float32, device=DEV)
    off_t = None if offsets is None else torch.from_numpy(np.asarray(offsets, np.int32)).to(DEV)
    cnt_t = None if count is None else torch.tensor([count], dtype=torch.int32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits), labels, out, offsets=off_t, count_dev=cnt_t)
    torch.cuda.synchronize()
    return out.cpu().numpy()[:n_out]


@pytest.mark.parametrize("rows,cols,dtype,std", [
    (4096, 10, torch.float32, 2.0), (1, 1, torch.float32, 1.0), (77, 2, torch.float32, 3.0),
    (1500, 100, torch.float32, 3.0), (700, 1000, torch.float32, 3.0), (301, 1001, torch.float32, 3.0),
    (257, 37, torch.bfloat16, 4.0), (129, 4095, torch.bfloat16, 4.0), (40, 8192, torch.bfloat16, 4.0),
    (67, 32000, torch.bfloat16, 4.0), (9, 32001, torch.bfloat16, 4.0), (5, 131072, torch.bfloat16, 4.0),
    (33, 2049, torch.float32, 3.0), (6, 70001, torch.float32, 5.0),
])
def test_row_losses(aa, rows, cols, dtype, std):
    logits = W.normal((rows, cols), std, rows + cols, dtype, DEV)
    labels = W.randint(0, cols, (rows,), rows * 7 + cols, DEV)
    got = run_loss(aa, logits, labels)
    ref = O.row_loss(W.to_oracle(logits), labels.cpu().numpy())
    assert np.max(np.abs(got - ref)) <= 1e-4, float(np.max(np.abs(got - ref)))


@pytest.mark.parametrize("rows,cols,dtype,pad", [
    (34001, 1000, torch.float32, 0), (17003, 4096, torch.bfloat16, 0), (33000, 1000, torch.float32, 24),
    (140000, 512, torch.bfloat16, 0), (350001, 100, torch.float32, 0),
])
def test_row_losses_on_large_inputs(aa, rows, cols, dtype, pad):
    """128 MB and more of logit rows of 0.4 to 8 KB: many rounds per CTA, strided rows, a device row count."""
    buf = W.normal((rows, cols + pad), 3.0, rows + cols, dtype, DEV)
    logits = buf[:, :cols]
    labels = W.randint(0, cols, (rows,), rows * 3 + cols, DEV)
    labels[5] = -1                                   # padding row
    count = rows - 3                                 # device-side row count: the last three rows stay untouched
    got = run_loss(aa, logits, labels, count=count)
    ref = O.row_loss(W.to_oracle(logits.contiguous()), labels.cpu().numpy())
    assert np.max(np.abs(got[:count] - ref[:count])) <= 1e-4, float(np.max(np.abs(got[:count] - ref[:count])))
    assert got[5] == 0.0 and np.all(got[count:] == -3.0)
    assert aa.aa_device_status() == B.AA_OK


def test_uniform_logits_give_ln_C_on_the_gpu(aa):
    for cols, dtype in ((10, torch.float32), (100, torch.float32), (1000, torch.float32), (32000, torch.bfloat16)):
        logits = torch.full((5, cols), 1.5, dtype=dtype, device=DEV)
        labels = W.randint(0, cols, (5,), 1, DEV)
        assert np.max(np.abs(run_loss(aa, logits, labels) - math.log(cols))) <= 1e-4


def test_loss_padding_bad_labels_masked_logits_strided_rows_and_device_count(aa):
    logits = W.normal((64, 50), 2.0, 5, torch.float32, DEV)
    logits[3, 10:20] = -float("inf")           # masked classes
    logits[4, :] = -float("inf"); logits[4, 7] = 0.5   # single live class
    labels = W.randint(0, 50, (64,), 6, DEV)
    labels[3] = 25; labels[4] = 7; labels[10] = -1; labels[11] = -100
    ref = O.row_loss(W.to_oracle(logits), labels.cpu().numpy())
    got = run_loss(aa, logits, labels)
    assert np.max(np.abs(got - ref)) <= 1e-4 and got[10] == 0.0 and got[11] == 0.0 and abs(got[4]) <= 1e-6
    assert aa.aa_device_status() == B.AA_OK
    labels[12] = 50                             # out of range: contributes 0 and latches
    got = run_loss(aa, logits, labels)
    assert got[12] == 0.0 and aa.aa_device_status() == B.AA_ERR_BAD_INDEX
    labels[12] = 0
    # row stride larger than cols
    wide = W.normal((40, 72), 2.0, 7, torch.bfloat16, DEV)
    view = wide[:, :65]
    ref = O.row_loss(W.to_oracle(view.contiguous()), labels[:40].cpu().numpy())
    assert np.max(np.abs(run_loss(aa, view, labels[:40].contiguous()) - ref)) <= 1e-4
    # device-side row count: rows beyond it are left untouched
    got = run_loss(aa, logits, labels, count=20)
    ref = O.row_loss(W.to_oracle(logits), labels.cpu().numpy())
    assert np.max(np.abs(got[:20] - ref[:20])) <= 1e-4 and np.all(got[20:] == -3.0)


@pytest.mark.parametrize("rows,cols,dtype", [(3000, 64, torch.float32), (700, 32000, torch.bfloat16)])
def test_per_sentence_sums(aa, rows, cols, dtype):
    logits = W.normal((rows, cols), 4.0, 21, dtype, DEV)
    labels = W.randint(0, cols, (rows,), 22, DEV)
    off = list(W.ragged_offsets(rows - 50, 8, 128, 23))   # last 50 rows belong to no sentence
    off = off[:3] + [off[3]] + off[3:]                    # one empty sentence
    got = run_loss(aa, logits, labels, offsets=off)
    ell = O.row_loss(W.to_oracle(logits), labels.cpu().numpy())
    ref = O.segment_sum(ell, off)
    tokens = np.maximum(1, np.diff(off))
    assert np.all(np.abs(got - ref) <= 1e-4 * tokens), float(np.max(np.abs(got - ref) / tokens))
    assert got[3] == 0.0
    # identity offsets reproduce the per-row losses; one segment gives the total
    ident = run_loss(aa, logits[:200], labels[:200].contiguous(), offsets=list(range(201)))
    assert np.max(np.abs(ident - ell[:200])) <= 1e-4
    total = run_loss(aa, logits[:200], labels[:200].contiguous(), offsets=[0, 200])
    assert abs(total[0] - ell[:200].sum()) <= 1e-4 * 200


# --------------------------------------------------------------------------
# Assistant step
# --------------------------------------------------------------------------

def assert_params_close(w_gpu, w_ref):
    w_ref = np.asarray(w_ref, np.float64)
    tol = 1e-4 * np.abs(w_ref) + 1e-4 * math.sqrt(float(np.mean(w_ref ** 2)) + 1e-300)
    err = np.abs(np.asarray(w_gpu, np.float64) - w_ref)
    assert np.all(err <= tol), float(np.max(err - tol))


@pytest.mark.parametrize("n,m,d,dtype,use_rows,thr", [
    (300, 300, 64, torch.float32, False, None), (5000, 2300, 64, torch.float32, True, None),
    (4000, 1777, 3072, torch.bfloat16, True, None), (900, 900, 100, torch.bfloat16, False, 2.0),
    (50, 1, 8, torch.float32, True, None), (600, 600, 7, torch.float32, False, 1.5),
    (400, 333, 4100, torch.float32, True, None), (2000, 2000, 512, torch.float32, False, None),
    (3000, 3000, 3072, torch.bfloat16, False, None), (1500, 700, 2048, torch.float32, True, 1.0),
    (900, 900, 2048, torch.bfloat16, False, None), (6000, 5000, 3072, torch.bfloat16, True, None),
])
def test_dense_assistant_step(aa, n, m, d, dtype, use_rows, thr):
    rng = np.random.default_rng(n + d)
    x = W.normal((n, d), 1.0, 60 + d, dtype, DEV)
    w = W.normal((d,), 0.05, 61, torch.float32, DEV)
    b = torch.full((1,), 0.3, device=DEV)
    loss = (W.normal((m,), 1.0, 62, torch.float32, DEV).abs() * 2).contiguous()
    rows = np.sort(rng.permutation(n)[:m]).astype(np.int32) if use_rows else None
    rows_t = None if rows is None else torch.from_numpy(rows).to(DEV)
    w0, b0 = w.cpu().numpy().copy(), float(b.item())
    feat = B.dense_features(x, row_idx=rows_t) if use_rows else B.dense_features(x[:m])
    cnt = torch.tensor([m], dtype=torch.int32, device=DEV)
    aa.aa_assistant_step(feat, loss, B.linear_assistant(w, b), 0.1, threshold=thr, count_dev=cnt)
    torch.cuda.synchronize()
    w_ref, b_ref, _ = O.assistant_step_linear_dense(W.to_oracle(x), loss.cpu().numpy(), w0, b0, 0.1, T=thr, row_idx=rows)
    assert_params_close(w.cpu().numpy(), w_ref)
    assert_params_close([b.item()], [b_ref] if abs(b_ref) > 0 else [1e-30])
    assert np.abs(w.cpu().numpy() - w0).max() > 0   # it did move


@pytest.mark.parametrize("n,m,d,mix", [(4000, None, 3072, 0.3), (9000, None, 1024, 0.1), (700, None, 256, 0.5)])
def test_dense_assistant_step_with_the_scores_of_the_screen(aa, n, m, d, mix):
    """Sequential schedule: the step takes the pre-activations that screening wrote under the same parameters instead of
    recomputing them.  Checked against the oracle given the same scores, against the oracle recomputing them, and
    against the library's own recomputing route."""
    x = W.normal((n, d), 1.0, 160 + d, torch.bfloat16, DEV)
    w = W.normal((d,), 0.03, 161, torch.float32, DEV)
    b = torch.full((1,), -0.2, device=DEV)
    asst = B.linear_assistant(w, b)
    out_idx = torch.zeros(n, dtype=torch.int32, device=DEV)
    cnt = torch.zeros(1, dtype=torch.int32, device=DEV)
    score = torch.zeros(n, dtype=torch.float32, device=DEV)
    aa.aa_score_shrink(B.dense_features(x), asst, mix, 3, 7, out_idx, cnt, score)
    torch.cuda.synchronize()
    mm = int(cnt.item())
    assert 0 < mm < n
    rows = out_idx.cpu().numpy()[:mm].astype(np.int32)
    loss = (W.normal((n,), 1.0, 162, torch.float32, DEV).abs() * 2).contiguous()
    w0, b0 = w.cpu().numpy().copy(), float(b.item())
    batch = B.dense_features(x, row_idx=out_idx)
    aa.aa_assistant_step_scored(batch, loss, score, asst, 0.1, count_dev=cnt)
    torch.cuda.synchronize()
    w_scored, b_scored = w.cpu().numpy().copy(), float(b.item())
    f = loss.cpu().numpy()[:mm]
    xh = W.to_oracle(x)
    # the oracle with the very scores the GPU used, and the oracle evaluating them itself
    w_given, b_given, _ = O.assistant_step_linear_dense(xh, f, w0, b0, 0.1, row_idx=rows, s=score.cpu().numpy()[rows])
    w_ref, b_ref, _ = O.assistant_step_linear_dense(xh, f, w0, b0, 0.1, row_idx=rows)
    for wr, br in ((w_given, b_given), (w_ref, b_ref)):
        assert_params_close(w_scored, wr)
        assert_params_close([b_scored], [br])
    # the recomputing route from the same starting point
    w.copy_(torch.from_numpy(w0)); b.fill_(b0)
    aa.aa_assistant_step(batch, loss, asst, 0.1, count_dev=cnt)
    torch.cuda.synchronize()
    assert_params_close(w.cpu().numpy(), w_ref)
    assert_params_close(w.cpu().numpy(), w_scored)
    assert np.abs(w_scored - w0).max() > 0


def test_assistant_step_empty_batch_and_zero_lr_leave_parameters_alone(aa):
    x = W.normal((100, 32), 1.0, 1, torch.float32, DEV)
    w = W.normal((32,), 0.1, 2, torch.float32, DEV)
    b = torch.full((1,), 0.5, device=DEV)
    w0 = w.clone()
    loss = torch.ones(100, device=DEV)
    zero = torch.zeros(1, dtype=torch.int32, device=DEV)
    aa.aa_assistant_step(B.dense_features(x), loss, B.linear_assistant(w, b), 0.5, count_dev=zero)
    aa.aa_assistant_step(B.dense_features(x), loss, B.linear_assistant(w, b), 0.0)
    torch.cuda.synchronize()
    assert torch.equal(w, w0) and b.item() == 0.5


def test_csr_assistant_step(aa):
    n, d, m = 3000, 1 << 14, 1200
    indptr, col, val = make_csr(n, d, 60, 70, empty_every=11)
    rng = np.random.default_rng(71)
    rows = np.sort(rng.permutation(n)[:m]).astype(np.int32)
    w = W.normal((d,), 0.05, 72, torch.float32, DEV)
    b = torch.full((1,), 0.1, device=DEV)
    loss = (W.normal((m,), 1.0, 73, torch.float32, DEV).abs() * 3).contiguous()
    w0 = w.cpu().numpy().copy()
    ti, tc, tv = (torch.from_numpy(a).to(DEV) for a in (indptr, col, val))
    feat = B.csr_features(ti, tc, tv, d, row_idx=torch.from_numpy(rows).to(DEV))
    aa.aa_assistant_step(feat, loss, B.linear_assistant(w, b), 0.2)
    torch.cuda.synchronize()
    w_ref, b_ref, _ = O.assistant_step_linear_csr(indptr, col, val, loss.cpu().numpy(), w0, 0.1, 0.2, row_idx=rows)
    assert_params_close(w.cpu().numpy(), w_ref)
    assert_params_close([b.item()], [b_ref])
    untouched = np.ones(d, bool)
    for r in rows:
        untouched[col[indptr[r]:indptr[r + 1]]] = False
    assert np.array_equal(w.cpu().numpy()[untouched], w0[untouched])   # only the batch's columns move


# --------------------------------------------------------------------------
# whole step, tiny reference configuration
# --------------------------------------------------------------------------

def test_tiny_reference_config_full_step(aa):
    cfg = W.TinyRef()
    t = cfg.make(DEV)
    w, b = t["w"].clone(), t["b"].clone()
    asst = B.linear_assistant(w, b)
    out_idx = torch.zeros(cfg.n, dtype=torch.int32, device=DEV)
    out_count = torch.zeros(1, dtype=torch.int32, device=DEV)
    out_mask = torch.zeros(cfg.n, dtype=torch.uint8, device=DEV)
    aa.aa_score_shrink(B.dense_features(t["x"]), asst, cfg.gamma, cfg.philox_seed, cfg.step, out_idx, out_count, None, out_mask)
    m = int(out_count.item())
    batch = out_idx[:m].long()
    logits_b = t["logits"][batch].contiguous()     # the Boss's outputs for the batch
    labels_b = t["labels"][batch].contiguous()
    loss = torch.zeros(cfg.n, dtype=torch.float32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits_b), labels_b, loss, count_dev=out_count)
    aa.aa_assistant_step(B.dense_features(t["x"], row_idx=out_idx), loss, asst, cfg.lr, count_dev=out_count)
    torch.cuda.synchronize()
    # oracle, driven by the GPU's own mask so that a tie-band flip cannot shift every later stage
    mask = out_mask.cpu().numpy()
    Bref = O.compact(mask)
    assert np.array_equal(out_idx.cpu().numpy()[:m], Bref)
    f_ref = O.row_loss(W.to_oracle(t["logits"])[Bref], t["labels"].cpu().numpy()[Bref])
    f_gpu = loss.cpu().numpy()[:m]
    assert np.max(np.abs(f_gpu - f_ref)) <= 1e-4
    w_ref, b_ref, z = O.assistant_step_linear_dense(W.to_oracle(t["x"]), f_gpu, t["w"].cpu().numpy(), 0.0, cfg.lr, row_idx=Bref)
    assert 0 < z.sum() < m
    assert_params_close(w.cpu().numpy(), w_ref)
    assert_params_close([b.item()], [b_ref])
    # the plain relative bound (1e-4 of the weight itself) on every weight that is not tiny
    w_gpu, w_r = w.cpu().numpy().astype(np.float64), np.asarray(w_ref, np.float64)
    big = np.abs(w_r) >= 0.1 * math.sqrt(float(np.mean(w_r ** 2)))
    assert big.sum() > cfg.d // 2 and np.all(np.abs(w_gpu - w_r)[big] <= 1e-4 * np.abs(w_r)[big])
    assert abs(b.item() - float(b_ref)) <= 1e-4 * abs(float(b_ref))
    assert aa.aa_launch_count() > 0


# --------------------------------------------------------------------------
# full-size image-classification shape, in the launch configuration the benchmark times
# --------------------------------------------------------------------------

def test_image_shape_full_pool(aa):
    cfg = W.ImageShape()
    x = cfg.pool(0, DEV)
    w, b = cfg.assistant(DEV)
    feat, asst = B.dense_features(x), B.linear_assistant(w, b)
    gpu = screen(aa, feat, asst, cfg.n, cfg.gamma, cfg.philox_seed, 17)
    idx, m, s, mask = gpu
    assert m == int(mask.sum()) and np.array_equal(idx[:m], np.nonzero(mask)[0])
    # oracle on a sample of rows spread over the pool (first/last tiles included)
    sample = np.unique(np.concatenate([np.arange(64), np.arange(cfg.n - 64, cfg.n),
                                       np.random.default_rng(3).integers(0, cfg.n, 1024)])).astype(np.int32)
    xs = W.to_oracle(x[torch.from_numpy(sample).long().to(DEV)])
    wh = w.cpu().numpy()
    s_ref = O.score_dense(xs, wh, 0.0)
    xn = np.linalg.norm(x[torch.from_numpy(sample).long().to(DEV)].double().cpu().numpy(), axis=1)
    assert np.all(np.abs(s[sample] - s_ref) <= 1e-5 * (np.abs(s_ref) + np.linalg.norm(wh) * xn))
    g = O.sigmoid(s_ref)
    p = O.accept_prob(g, cfg.gamma)
    c = O.uniform(cfg.philox_seed, 17, sample)
    keep = O.shrink(g, cfg.gamma, cfg.philox_seed, 17, row_idx=sample)
    far = np.abs(p - c) >= 1e-5
    assert np.array_equal(mask[sample][far], keep[far])
    # acceptance statistics over the whole pool from the GPU's own (verified) scores
    p_all = O.accept_prob(O.sigmoid(s.astype(np.float64)), cfg.gamma)
    assert abs(m - p_all.sum()) < 5 * math.sqrt((p_all * (1 - p_all)).sum())


# --------------------------------------------------------------------------
# losses of a batch list out of logits stored for the whole pool
# --------------------------------------------------------------------------

@pytest.mark.parametrize("rows,cols,dtype,m", [
    (3000, 100, torch.float32, 1700), (517, 1000, torch.float32, 517), (300, 8200, torch.bfloat16, 120),
    (64, 33000, torch.bfloat16, 40), (1, 5, torch.float32, 1),
])
def test_instance_loss_of_listed_rows(aa, rows, cols, dtype, m):
    rng = np.random.default_rng(rows + cols)
    lg = W.normal((rows, cols), 3.0, 41 + rows, dtype, DEV)
    y = W.randint(0, cols, (rows,), 43 + rows, DEV).to(torch.int32)
    y[rows // 2] = -1                                                   # a padding row: loss 0
    listed = rng.integers(0, rows, m).astype(np.int32)                  # any order, repeats allowed
    if m > 2:
        listed[1] = rows // 2
    idx = torch.from_numpy(listed).to(DEV)
    out = torch.full((m + 3,), -5.0, dtype=torch.float32, device=DEV)
    # the device count cuts the list short; entries at and beyond it stay untouched
    m_dev = max(1, m - 2)
    cnt = torch.tensor([m_dev], dtype=torch.int32, device=DEV)
    aa.aa_instance_loss_rows(B.logits_desc(lg), y, idx, out, count_dev=cnt, n_rows=m)
    torch.cuda.synchronize()
    ref = O.instance_loss_rows(W.to_oracle(lg), y.cpu().numpy(), listed[:m_dev])
    got = out.cpu().numpy()
    assert np.all(np.abs(got[:m_dev] - ref) <= 1e-4)
    if m_dev > 1 and m > 2:
        assert got[1] == 0.0
    assert np.all(got[m_dev:] == -5.0)


def test_instance_loss_rows_bad_entry_latches_and_gives_zero():
    ctx = B.AutoAssist(max_rows=1024, max_d=16, device=DEV)
    lg = W.normal((100, 10), 1.0, 5, torch.float32, DEV)
    y = torch.zeros(100, dtype=torch.int32, device=DEV)
    idx = torch.tensor([3, 100, -1, 99], dtype=torch.int32, device=DEV)
    out = torch.full((4,), -5.0, dtype=torch.float32, device=DEV)
    ctx.aa_instance_loss_rows(B.logits_desc(lg), y, idx, out)
    assert ctx.aa_device_status() == B.AA_ERR_BAD_INDEX
    got = out.cpu().numpy()
    assert got[1] == 0.0 and got[2] == 0.0 and got[0] > 0 and got[3] > 0
    assert ctx.aa_device_status() == B.AA_OK
    ctx.close()


# --------------------------------------------------------------------------
# short aligned rows (the register-resident loss kernel): widths at and around its limits, extreme logits
# --------------------------------------------------------------------------

@pytest.mark.parametrize("rows,cols,dtype", [
    (5000, 4, torch.float32), (333, 8, torch.float32), (2049, 16, torch.float32), (4100, 100, torch.float32),
    (1000, 128, torch.float32), (1000, 132, torch.float32), (777, 8, torch.bfloat16), (1025, 64, torch.bfloat16),
    (3000, 256, torch.bfloat16), (500, 264, torch.bfloat16), (1, 32, torch.float32),
])
def test_short_row_losses(aa, rows, cols, dtype):
    logits = W.normal((rows, cols), 3.0, rows + 3 * cols, dtype, DEV)
    labels = W.randint(0, cols, (rows,), rows + cols, DEV)
    if rows > 10:
        labels[3] = -1                                    # padding row
        logits[5] = 80.0 if dtype == torch.float32 else 64.0     # all equal and large: loss = ln(cols)
        logits[7, :] = -1e30 if dtype == torch.float32 else -3e38  # one finite winner among hugely negative logits
        logits[7, cols - 1] = 2.0
        labels[7] = cols - 1
    count = rows if rows < 10 else rows - 4                   # the device count cuts the last rows off
    out = torch.full((rows,), -3.0, dtype=torch.float32, device=DEV)
    cnt_t = torch.tensor([count], dtype=torch.int32, device=DEV)
    aa.aa_instance_loss(B.logits_desc(logits), labels, out, count_dev=cnt_t)
    torch.cuda.synchronize()
    got = out.cpu().numpy()
    ref = O.row_loss(W.to_oracle(logits), labels.cpu().numpy())
    assert np.max(np.abs(got[:count] - ref[:count])) <= 1e-4, float(np.max(np.abs(got[:count] - ref[:count])))
    assert np.all(got[count:] == -3.0)
    if rows > 10:
        assert got[3] == 0.0 and abs(got[5] - math.log(cols)) <= 1e-4 and abs(got[7]) <= 1e-6
