"""Pins of the CPU oracle against things other than itself.

Each test fixes the oracle to a value the paper, the mathematics or an
independent library fixes: cuRAND's host Philox generator, a separate NumPy
restatement of Philox, closed forms, brute force in extended precision,
torch's float64 cross-entropy, finite differences of the Assistant objective,
and the literal sequential loop of Algorithm 1.
"""
import ctypes
import math
import os

import numpy as np
import pytest
import torch

from oracle import aa_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        line = line.strip()
        if line and not line.startswith("#"):
            k, v = line.split()
            out[k] = float(v)
    return out


# --------------------------------------------------------------------------
# Philox4x32-10
# --------------------------------------------------------------------------

def _curand():
    for path in ("/usr/local/cuda/lib64/libcurand.so.10", "libcurand.so.10", "libcurand.so"):
        try:
            return ctypes.CDLL(path)
        except OSError:
            continue
    try:
        import nvidia.curand

        base = os.path.join(os.path.dirname(nvidia.curand.__file__), "lib")
        for f in os.listdir(base):
            if f.startswith("libcurand.so"):
                return ctypes.CDLL(os.path.join(base, f))
    except Exception:
        pass
    return None


def _curand_words(lib, seed, offset, n):
    gen = ctypes.c_void_p()
    assert lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) == 0  # CURAND_RNG_PSEUDO_PHILOX4_32_10
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    assert lib.curandSetGeneratorOffset(gen, ctypes.c_ulonglong(offset)) == 0
    out = np.zeros(n, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(n)) == 0
    lib.curandDestroyGenerator(gen)
    return out


@pytest.mark.parametrize("seed", [0, 1, 0x9F3A5C7E12345678])
@pytest.mark.parametrize("block", [0, 3, (1 << 32) + 5])
def test_philox_matches_curand_host_generator(seed, block):
    """cuRAND's host generator: seed -> key; in its default ordering output block q (four
    words) comes from subsequence q mod 65536 (counter words 2-3) at position q div 65536
    (counter words 0-1), so one call pins the key and every counter position."""
    lib = _curand()
    if lib is None:
        pytest.skip("libcurand not found")
    words = _curand_words(lib, seed, 4 * block * 65536, 32)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    for sub in range(8):
        ref = O.philox4x32_10([block & 0xFFFFFFFF, block >> 32, sub, 0], key)
        assert [int(v) for v in ref] == [int(v) for v in words[4 * sub:4 * sub + 4]]


def _philox_numpy(ctr, key):
    """Independent vectorised restatement (uint64 arithmetic) of Philox4x32-10."""
    c = [np.asarray(v, dtype=np.uint64) for v in ctr]
    k = [np.asarray(v, dtype=np.uint64) for v in key]
    mask = np.uint64(0xFFFFFFFF)
    for _ in range(10):
        prod_a = np.uint64(0xD2511F53) * c[0]
        prod_b = np.uint64(0xCD9E8D57) * c[2]
        c = [((prod_b >> np.uint64(32)) ^ c[1] ^ k[0]) & mask, prod_b & mask,
             ((prod_a >> np.uint64(32)) ^ c[3] ^ k[1]) & mask, prod_a & mask]
        k = [(k[0] + np.uint64(0x9E3779B9)) & mask, (k[1] + np.uint64(0xBB67AE85)) & mask]
    return [v.astype(np.uint32) for v in c]


def test_philox_matches_numpy_restatement_on_all_counter_words():
    rng = np.random.default_rng(11)
    ctr = rng.integers(0, 1 << 32, size=(4, 256), dtype=np.uint64)
    key = rng.integers(0, 1 << 32, size=(2, 256), dtype=np.uint64)
    ref = _philox_numpy(list(ctr), list(key))
    for t in range(256):
        got = O.philox4x32_10(ctr[:, t], key[:, t])
        assert [int(v) for v in got] == [int(ref[j][t]) for j in range(4)]


def test_uniform_keying_and_range():
    """c = top 24 bits of word 0 at counter (id, step), key = seed."""
    seed, step = 0x0123456789ABCDEF, (7 << 32) + 3
    ids = np.array([0, 1, 5, (1 << 32) + 9], dtype=np.uint64)
    u = O.uniform(seed, step, ids)
    for i, ui in zip(ids, u):
        i = int(i)
        words = _philox_numpy([i & 0xFFFFFFFF, i >> 32, step & 0xFFFFFFFF, step >> 32],
                              [seed & 0xFFFFFFFF, seed >> 32])
        assert ui == float(int(words[0]) >> 8) / float(1 << 24)
        assert 0.0 <= ui < 1.0
        assert np.float32(ui) == ui  # exact in fp32


def test_uniform_statistics_and_stream_separation():
    n = 200_000
    ids = np.arange(n)
    u0 = O.uniform(0, 0, ids)
    u1 = O.uniform(0, 1, ids)
    u2 = O.uniform(1, 0, ids)
    for u in (u0, u1, u2):
        assert abs(u.mean() - 0.5) < 5 * math.sqrt(1 / 12 / n)
        assert abs(u.var() - 1 / 12) < 5 * math.sqrt(1 / 180 / n)
        hist = np.bincount((u * 256).astype(int), minlength=256)
        chi2 = ((hist - n / 256) ** 2 / (n / 256)).sum()
        assert chi2 < 255 + 6 * math.sqrt(2 * 255)
    lim = 5 / math.sqrt(n)
    assert abs(np.corrcoef(u0[:-1], u0[1:])[0, 1]) < lim   # across ids
    assert abs(np.corrcoef(u0, u1)[0, 1]) < lim            # across steps
    assert abs(np.corrcoef(u0, u2)[0, 1]) < lim            # across seeds


# --------------------------------------------------------------------------
# Scores, g, acceptance probability
# --------------------------------------------------------------------------

def test_zero_weights_give_the_closed_form_probability():
    x = np.random.default_rng(0).standard_normal((37, 19)).astype(np.float32)
    s = O.score_dense(x, np.zeros(19, np.float32), 0.0)
    assert np.all(s == 0.0)
    g = O.sigmoid(s)
    assert np.all(g == 0.5)
    gold = golden()
    for gamma in (0.1, 0.2, 0.05, 0.5):
        assert np.allclose(O.accept_prob(g, gamma), gold[f"accept_prob_zero_weights_gamma_{gamma}"], atol=1e-15)


def test_score_is_the_inner_product_one_hot_and_bias():
    d = 23
    w = np.random.default_rng(1).standard_normal(d).astype(np.float32)
    x = np.eye(d, dtype=np.float32)
    s = O.score_dense(x, w, 0.25)
    assert np.array_equal(s, w.astype(np.float64) + 0.25)
    # a wrong stride or transposed operand fails this: non-square, distinct entries
    x2 = np.arange(3 * d, dtype=np.float32).reshape(3, d) / 7
    expect = [math.fsum(float(a) * float(b) for a, b in zip(row, w)) - 1.5 for row in x2]
    assert np.allclose(O.score_dense(x2, w, -1.5), expect, rtol=1e-14, atol=1e-12)
    # gather list
    assert np.array_equal(O.score_dense(x2, w, 0.0, row_idx=[2, 0]), O.score_dense(x2, w, 0.0)[[2, 0]])


def test_bf16_rows_are_widened_exactly():
    t = torch.tensor([[1.0, -2.5, 0.33203125], [3.0, 0.0078125, -0.5]], dtype=torch.bfloat16)
    bits = t.view(torch.int16).numpy().view(np.uint16)
    w = np.array([2.0, 4.0, 8.0], np.float32)
    assert np.array_equal(O.score_dense(bits, w, 0.0), (t.double().numpy() * w).sum(1))


def test_csr_score_equals_dense_score_with_duplicates():
    rng = np.random.default_rng(2)
    n, d = 41, 30
    dense = np.zeros((n, d), np.float32)
    indptr, col, val = [0], [], []
    for i in range(n):
        k = int(rng.integers(0, 9))        # empty rows included
        cols = rng.integers(0, d, k)       # duplicates allowed
        vals = rng.integers(1, 4, k).astype(np.float32)
        for c, v in zip(cols, vals):
            dense[i, c] += v
        col += list(cols); val += list(vals); indptr.append(len(col))
    w = rng.standard_normal(d).astype(np.float32)
    a = O.score_csr(indptr, np.array(col, np.int32), np.array(val, np.float32), w, 0.5)
    b = O.score_dense(dense, w, 0.5)
    assert np.allclose(a, b, rtol=1e-13, atol=1e-13)


def test_sigmoid_symmetry_and_extremes():
    s = np.array([-800.0, -30.0, -1.0, 0.0, 1.0, 30.0, 800.0])
    g = O.sigmoid(s)
    assert np.all(np.isfinite(g)) and g[0] == 0.0 and g[-1] == 1.0 and g[3] == 0.5
    assert np.allclose(g + g[::-1], 1.0, atol=1e-16)
    assert np.allclose(g[4], 1 / (1 + math.exp(-1.0)), rtol=1e-15)


def test_mlp_score_reduces_to_known_cases():
    rng = np.random.default_rng(3)
    n, d = 9, 6
    x = rng.standard_normal((n, d)).astype(np.float32)
    # selector W1 = I, w2 = 1: s = sum_j relu(x_j)
    s = O.score_mlp(x, np.eye(d), np.zeros(d), np.ones(d), 0.0)
    assert np.allclose(s, np.maximum(x.astype(np.float64), 0).sum(1), rtol=1e-15)
    # one hidden unit, positive inputs and weights: equals the linear score scaled by w2
    xp = np.abs(x) + 0.1
    w = np.abs(rng.standard_normal(d)) + 0.1
    s1 = O.score_mlp(xp.astype(np.float32), w[None, :], np.array([0.3]), np.array([2.0]), -1.0)
    assert np.allclose(s1, 2.0 * (O.score_dense(xp.astype(np.float32), w, 0.3)) - 1.0, rtol=1e-14)
    # non-square W1 with distinct entries against explicit loops (catches a transposed W1)
    W1 = rng.standard_normal((4, d)); b1 = rng.standard_normal(4); w2 = rng.standard_normal(4)
    s2, a2 = O.score_mlp(x, W1, b1, w2, 0.7, want_pre=True)
    for i in range(n):
        pre = [math.fsum(W1[u, j] * float(x[i, j]) for j in range(d)) + b1[u] for u in range(4)]
        assert np.allclose(a2[i], pre, rtol=1e-13, atol=1e-13)
        assert math.isclose(s2[i], 0.7 + sum(w2[u] * max(pre[u], 0.0) for u in range(4)), rel_tol=1e-12, abs_tol=1e-12)


# --------------------------------------------------------------------------
# Algorithm 1: shrink decision and ordered batch
# --------------------------------------------------------------------------

def test_two_branch_rule_equals_single_compare_away_from_ties():
    rng = np.random.default_rng(4)
    n = 50_000
    g = rng.random(n)
    for gamma in (0.0, 0.05, 0.1, 0.2, 0.5, 0.9):
        keep = O.shrink(g, gamma, seed=3, step=9)
        c = O.uniform(3, 9, np.arange(n))
        p = O.accept_prob(g, gamma)
        far = np.abs(c - p) > 1e-12
        assert np.array_equal(keep[far].astype(bool), (c < p)[far])


def test_gamma_extremes():
    n = 5000
    g = np.random.default_rng(5).random(n)
    assert np.all(O.shrink(g, 1.0, 0, 0) == 1)                          # floor accepts everything
    assert np.array_equal(O.compact(O.shrink(g, 1.0, 0, 0)), np.arange(n, dtype=np.int32))
    c = O.uniform(0, 0, np.arange(n))
    assert np.array_equal(O.shrink(g, 0.0, 0, 0).astype(bool), c < g)   # pure Bernoulli(g)
    assert np.all(O.shrink(np.ones(n), 0.0, 0, 0) == 1)                 # p = 1 always keeps (c < 1)
    assert np.all(O.shrink(np.zeros(n), 0.0, 0, 0) == 0)                # p = 0 never keeps


def test_acceptance_count_is_consistent_with_the_probabilities():
    rng = np.random.default_rng(6)
    n = 100_000
    g = O.sigmoid(rng.standard_normal(n) * 2)
    for gamma, step in ((0.1, 0), (0.2, 1), (0.5, 2)):
        p = O.accept_prob(g, gamma)
        keep = O.shrink(g, gamma, 0, step)
        sd = math.sqrt((p * (1 - p)).sum())
        assert abs(keep.sum() - p.sum()) < 5 * sd
        # calibration per decile of p
        order = np.argsort(p)
        for chunk in np.array_split(order, 10):
            sdc = math.sqrt((p[chunk] * (1 - p[chunk])).sum())
            assert abs(keep[chunk].sum() - p[chunk].sum()) < 5 * sdc


def test_compaction_is_nonzero_of_the_mask_in_order():
    rng = np.random.default_rng(7)
    for n in (0, 1, 2, 31, 32, 33, 1000):
        keep = (rng.random(n) < 0.4).astype(np.uint8)
        B = O.compact(keep)
        assert np.array_equal(B, np.nonzero(keep)[0].astype(np.int32))
        assert len(B) == int(keep.sum())
        assert np.all(np.diff(B) > 0)
    perm = rng.permutation(1000).astype(np.int32)
    keep = (rng.random(1000) < 0.4).astype(np.uint8)
    assert np.array_equal(O.compact(keep, row_idx=perm), perm[np.nonzero(keep)[0]])


def test_sequential_algorithm_1_is_a_prefix_of_the_ordered_survivors():
    rng = np.random.default_rng(8)
    n = 4000
    g = rng.random(n)
    perm = rng.permutation(n).astype(np.int32)
    for row_idx in (None, perm):
        full = O.compact(O.shrink(g, 0.15, 21, 4, id_base=100, row_idx=row_idx), row_idx=row_idx)
        for bs in (1, 7, 64, len(full), len(full) + 50):
            B, consumed = O.sample_batch(g, 0.15, 21, 4, bs, id_base=100, row_idx=row_idx)
            assert np.array_equal(B, full[:bs])
            if bs <= len(full):
                rows = perm if row_idx is not None else np.arange(n)
                assert rows[consumed - 1] == full[bs - 1]   # stopped right after the bs-th accept
            else:
                assert consumed == n


# --------------------------------------------------------------------------
# Boss loss per instance
# --------------------------------------------------------------------------

@pytest.mark.parametrize("C", [1, 2, 10, 100, 1000, 32000])
def test_uniform_logits_give_ln_C(C):
    logits = np.full((3, C), 1.75, np.float32)
    ell = O.row_loss(logits, np.array([0, C // 2, C - 1], np.int32))
    assert np.allclose(ell, math.log(C), rtol=0, atol=1e-12)


def test_row_loss_against_long_double_brute_force():
    rng = np.random.default_rng(9)
    logits = (rng.standard_normal((64, 13)) * 2).astype(np.float32)
    labels = rng.integers(0, 13, 64).astype(np.int32)
    ell = O.row_loss(logits, labels)
    ld = logits.astype(np.longdouble)
    brute = np.log(np.exp(ld).sum(1)) - ld[np.arange(64), labels]
    assert np.allclose(ell, brute.astype(np.float64), rtol=0, atol=1e-13)


def test_row_loss_matches_torch_float64_cross_entropy():
    rng = np.random.default_rng(10)
    logits = (rng.standard_normal((200, 77)) * 4).astype(np.float32)
    labels = rng.integers(0, 77, 200).astype(np.int32)
    ref = torch.nn.functional.cross_entropy(torch.from_numpy(logits).double(),
                                            torch.from_numpy(labels).long(), reduction="none").numpy()
    assert np.allclose(O.row_loss(logits, labels), ref, rtol=0, atol=1e-12)
    # bf16 storage: same check on the widened values
    t = torch.from_numpy(logits).to(torch.bfloat16)
    ref16 = torch.nn.functional.cross_entropy(t.double(), torch.from_numpy(labels).long(), reduction="none").numpy()
    assert np.allclose(O.row_loss(t.view(torch.int16).numpy().view(np.uint16), labels), ref16, rtol=0, atol=1e-12)


def test_row_loss_properties():
    rng = np.random.default_rng(12)
    logits = (rng.standard_normal((50, 9)) * 3).astype(np.float32)
    labels = rng.integers(0, 9, 50).astype(np.int32)
    base = O.row_loss(logits, labels)
    assert np.allclose(O.row_loss(logits + np.float32(8.0), labels), base, atol=1e-5)   # shift invariance
    # two classes: softplus of the gap
    two = np.array([[0.3, -1.2], [2.0, 5.0]], np.float32)
    assert np.allclose(O.row_loss(two, [0, 0]), [math.log1p(math.exp(-1.5)), math.log1p(math.exp(3.0))], atol=1e-7)
    # dominant logit: ~0 when it is the label, ~gap otherwise
    dom = np.zeros((2, 6), np.float32); dom[:, 2] = 60.0
    out = O.row_loss(dom, [2, 4])
    assert out[0] < 1e-20 + 1e-12 and abs(out[1] - 60.0) < 1e-12
    # huge magnitudes stay finite (max subtraction), -inf entries are masked
    big = np.array([[1e30, -1e30, 0.0], [-np.inf, 0.0, 0.0]], np.float32)
    out = O.row_loss(big, [0, 1])
    assert out[0] == 0.0 and abs(out[1] - math.log(2)) < 1e-15
    # padding (negative label) and out-of-range labels contribute 0
    assert np.array_equal(O.row_loss(logits[:2], [-1, 9]), [0.0, 0.0])


def test_segment_sums():
    rng = np.random.default_rng(13)
    ell = rng.random(40)
    assert np.array_equal(O.segment_sum(ell, np.arange(41)), ell)                      # identity offsets
    assert math.isclose(O.segment_sum(ell, [0, 40])[0], math.fsum(ell), rel_tol=1e-14)  # one segment
    off = [0, 3, 3, 17, 40]                                                            # empty segment -> 0
    L = O.segment_sum(ell, off)
    assert L[1] == 0.0
    assert np.allclose(L, [math.fsum(ell[a:b]) for a, b in zip(off[:-1], off[1:])], rtol=1e-14)
    assert math.isclose(L.sum(), math.fsum(ell), rel_tol=1e-13)                        # additivity


# --------------------------------------------------------------------------
# Labels, objective, gradient, update
# --------------------------------------------------------------------------

def test_label_rule_is_strict_and_batch_mean():
    gold = golden()
    f = np.full(100, 2.5, np.float32)
    assert O.labels(f, O.batch_mean(f)).sum() == gold["labels_constant_loss_positive_count"]
    f2 = np.array([1.0, 3.0, 1.0, 3.0, 3.0], np.float32)
    assert O.batch_mean(f2) == 2.2
    assert np.array_equal(O.labels(f2, O.batch_mean(f2)), [0, 1, 0, 1, 1])
    assert np.array_equal(O.labels(f2, 3.0), [0, 0, 0, 0, 0])     # f > T, not >=
    assert O.batch_mean(np.zeros(0, np.float32)) == 0.0


def test_objective_closed_forms():
    gold = golden()
    z = np.array([0, 1, 1, 0, 1], np.uint8)
    assert math.isclose(O.bce_mean(np.zeros(5), z), gold["bce_zero_weights"], rel_tol=1e-15)
    s = np.array([0.7, -1.3, 2.0, 12.0, -12.0])   # the direct form below loses g = 1 beyond |s| ~ 36
    g = 1 / (1 + np.exp(-s))
    direct = -(z * np.log(g) + (1 - z) * np.log1p(-g)).mean()
    assert math.isclose(O.bce_mean(s, z), direct, rel_tol=1e-10)
    # far tails: BCE -> |s| on the wrong side, 0 on the right side
    assert math.isclose(O.bce_mean(np.array([800.0, -800.0, 800.0]), np.array([0, 1, 1], np.uint8)), 1600.0 / 3)


def _fd(fun, theta, h=1e-6):
    out = np.zeros_like(theta)
    flat, of = theta.reshape(-1), out.reshape(-1)
    for j in range(flat.size):
        keep = flat[j]
        flat[j] = keep + h; up = fun()
        flat[j] = keep - h; dn = fun()
        flat[j] = keep
        of[j] = (up - dn) / (2 * h)
    return out


def test_linear_gradient_matches_finite_differences_dense_and_csr():
    rng = np.random.default_rng(14)
    m, d = 17, 7
    x = rng.standard_normal((m + 3, d)).astype(np.float32)
    rows = rng.permutation(m + 3)[:m].astype(np.int32)
    z = rng.integers(0, 2, m).astype(np.uint8)
    w = rng.standard_normal(d) * 0.5
    bb = np.array([0.2])
    obj = lambda: O.bce_mean(O.score_dense(x, w, bb[0], row_idx=rows), z)
    gw, gb = O.linear_grad_dense(x, O.score_dense(x, w, bb[0], row_idx=rows), z, row_idx=rows)
    assert np.allclose(gw, _fd(obj, w), rtol=1e-6, atol=1e-9)
    assert np.allclose(gb, _fd(obj, bb)[0], rtol=1e-6, atol=1e-9)
    # CSR with duplicate columns
    indptr, col, val = [0], [], []
    for i in range(m):
        k = int(rng.integers(0, 6)); col += list(rng.integers(0, d, k)); val += list(rng.random(k) + 0.5)
        indptr.append(len(col))
    col, val = np.array(col, np.int32), np.array(val, np.float32)
    obj2 = lambda: O.bce_mean(O.score_csr(indptr, col, val, w, bb[0]), z)
    gw2, gb2 = O.linear_grad_csr(indptr, col, val, d, O.score_csr(indptr, col, val, w, bb[0]), z)
    assert np.allclose(gw2, _fd(obj2, w), rtol=1e-6, atol=1e-9)
    assert np.allclose(gb2, _fd(obj2, bb)[0], rtol=1e-6, atol=1e-9)


def test_mlp_gradient_matches_finite_differences():
    rng = np.random.default_rng(15)
    m, d, hdim = 11, 5, 4
    x = rng.standard_normal((m, d)).astype(np.float32)
    z = rng.integers(0, 2, m).astype(np.uint8)
    W1 = rng.standard_normal((hdim, d)) * 0.7
    b1 = rng.standard_normal(hdim) * 0.3
    w2 = rng.standard_normal(hdim)
    b2 = np.array([0.1])
    obj = lambda: O.bce_mean(O.score_mlp(x, W1, b1, w2, b2[0]), z)
    s, a = O.score_mlp(x, W1, b1, w2, b2[0], want_pre=True)
    assert np.min(np.abs(a)) > 1e-4   # no unit sits on the ReLU kink within the FD step
    gW1, gb1, gw2, gb2 = O.mlp_grad(x, a, s, z, w2)
    assert np.allclose(gW1, _fd(obj, W1), rtol=1e-6, atol=1e-9)
    assert np.allclose(gb1, _fd(obj, b1), rtol=1e-6, atol=1e-9)
    assert np.allclose(gw2, _fd(obj, w2), rtol=1e-6, atol=1e-9)
    assert np.allclose(gb2, _fd(obj, b2)[0], rtol=1e-6, atol=1e-9)


def test_update_special_cases():
    # one instance, x = e_j: only w_j and b move, by -lr (sigma(w_j + b) - z)
    d, j = 6, 4
    w = np.linspace(-0.5, 0.5, d).astype(np.float32)
    b = np.float32(0.25)
    x = np.zeros((1, d), np.float32); x[0, j] = 1.0
    f = np.array([5.0], np.float32)
    w1, b1, z = O.assistant_step_linear_dense(x, f, w, b, lr=0.5, T=1.0)
    assert z[0] == 1
    delta = -0.5 * (1 / (1 + math.exp(-(float(w[j]) + 0.25))) - 1.0)
    expect = w.copy(); expect[j] = np.float32(float(w[j]) + delta)
    assert np.array_equal(w1, expect)
    assert b1 == np.float32(0.25 + delta)
    # handing in the pre-activation replaces the dot product and nothing else: s = 0 gives sigma = 1/2 whatever w is
    w1s, b1s, _ = O.assistant_step_linear_dense(x, f, w, b, lr=0.5, T=1.0, s=np.array([0.0]))
    expect_s = w.copy(); expect_s[j] = np.float32(float(w[j]) - 0.5 * (0.5 - 1.0))
    assert np.array_equal(w1s, expect_s) and b1s == np.float32(0.25 - 0.5 * (0.5 - 1.0))
    w1e, b1e, _ = O.assistant_step_linear_dense(x, f, w, b, lr=0.5, T=1.0, s=np.array([float(w[j]) + 0.25]))
    assert np.array_equal(w1e, w1) and b1e == b1
    # lr = 0 and empty batch leave the parameters unchanged
    w2, b2, _ = O.assistant_step_linear_dense(x, f, w, b, lr=0.0, T=1.0)
    assert np.array_equal(w2, w) and b2 == b
    w3, b3, _ = O.assistant_step_linear_dense(x, np.zeros(0, np.float32), w, b, lr=0.5)
    assert np.array_equal(w3, w) and b3 == b


def test_composed_csr_step_special_cases():
    """assistant_step_linear_csr chains labels, score_csr, linear_grad_csr and sgd: pinned on the one-instance closed
    form (a count of c in bucket j moves w_j by -lr c (sigma(c w_j + b) - z) and b by -lr (sigma(c w_j + b) - z), and
    nothing else), on a batch list that selects that one row out of several, and against the dense twin."""
    d, j, c = 7, 2, 3.0
    w = np.linspace(-0.4, 0.6, d).astype(np.float32)
    b = np.float32(-0.15)
    # three stored rows; the batch is row 1 alone: bucket j with count c (stored as one entry of value c)
    indptr = np.array([0, 2, 3, 5], np.int32)
    col = np.array([0, 5, j, 1, 6], np.int32)
    val = np.array([1.0, 2.0, c, 1.0, 1.0], np.float32)
    f = np.array([0.3], np.float32)
    w1, b1, z = O.assistant_step_linear_csr(indptr, col, val, f, w, b, lr=0.25, T=1.0, row_idx=np.array([1], np.int32))
    assert z[0] == 0
    r = 1.0 / (1.0 + math.exp(-(c * float(w[j]) + float(b))))            # sigma(s) - 0
    expect = w.copy(); expect[j] = np.float32(float(w[j]) - 0.25 * c * r)
    assert np.array_equal(w1, expect)
    assert b1 == np.float32(float(b) - 0.25 * r)
    # batch mean threshold over two instances with different losses: exactly the larger one is labelled 1
    f2 = np.array([0.2, 0.9], np.float32)
    _, _, z2 = O.assistant_step_linear_csr(indptr, col, val, f2, w, b, lr=0.1, row_idx=np.array([0, 2], np.int32))
    assert list(z2) == [0, 1]
    # n_cand: only the first len(f) entries of a longer batch list are used
    wa, ba, _ = O.assistant_step_linear_csr(indptr, col, val, f, w, b, lr=0.25, T=1.0, row_idx=np.array([1, 0, 2], np.int32))
    assert np.array_equal(wa, w1) and ba == b1
    # the dense twin on the densified rows takes the same step (repeated buckets add)
    rng = np.random.default_rng(21)
    n, d2 = 30, 12
    lens = rng.integers(0, 6, n)
    ip = np.zeros(n + 1, np.int32); ip[1:] = np.cumsum(lens)
    cc = rng.integers(0, d2, int(ip[-1])).astype(np.int32)
    vv = rng.integers(1, 4, int(ip[-1])).astype(np.float32)
    dense = np.zeros((n, d2), np.float32)
    for i in range(n):
        for k in range(ip[i], ip[i + 1]):
            dense[i, cc[k]] += vv[k]
    w0 = (rng.normal(size=d2) * 0.3).astype(np.float32)
    rows = np.sort(rng.permutation(n)[:17]).astype(np.int32)
    ff = np.abs(rng.normal(size=17)).astype(np.float32)
    wc, bc, zc = O.assistant_step_linear_csr(ip, cc, vv, ff, w0, 0.2, lr=0.3, row_idx=rows)
    wd, bd, zd = O.assistant_step_linear_dense(dense, ff, w0, 0.2, lr=0.3, row_idx=rows)
    assert np.array_equal(zc, zd) and np.allclose(wc, wd, rtol=0, atol=1e-7) and abs(float(bc) - float(bd)) <= 1e-7
    # lr = 0 and an empty batch leave the parameters unchanged
    w3, b3, _ = O.assistant_step_linear_csr(indptr, col, val, f, w, b, lr=0.0, T=1.0, row_idx=np.array([1], np.int32))
    assert np.array_equal(w3, w) and b3 == b
    w4, b4, _ = O.assistant_step_linear_csr(indptr, col, val, np.zeros(0, np.float32), w, b, lr=0.5)
    assert np.array_equal(w4, w) and b4 == b


def test_conv_pool_features_reduce_to_known_forms_and_match_torch():
    """The convolutional Assistant's feature map (convolution with the Boss's weights, rectifier, average pooling) is
    pinned on closed forms and on torch's float64 conv2d / avg_pool2d (library routines, not the oracle's own loops)."""
    rng = np.random.default_rng(31)
    n, c_in, H, Wd = 3, 3, 8, 8
    x = rng.random((n, c_in * H * Wd)).astype(np.float32)                   # non-negative pixels
    # identity taps (centre 1, channel c -> channel c), no bias, global average pooling: phi = per-channel mean pixel,
    # so the linear head on phi is the linear Assistant on the pooled pixels
    ident = np.zeros((c_in, c_in, 3, 3)); ident[np.arange(c_in), np.arange(c_in), 1, 1] = 1.0
    phi = O.conv_pool_features(x, c_in, H, Wd, ident, np.zeros(c_in), pool=8)
    assert phi.shape == (n, c_in)
    assert np.allclose(phi, x.reshape(n, c_in, -1).astype(np.float64).mean(axis=2), rtol=0, atol=1e-15)
    head = rng.normal(size=c_in)
    assert np.allclose(phi @ head + 0.5, O.score_dense(phi.astype(np.float32), head, 0.5), atol=1e-6)
    # zero taps: phi = relu(bias) everywhere, whatever the pooling
    bias = np.array([0.7, -0.3, 0.0, 1.5])
    phi0 = O.conv_pool_features(x, c_in, H, Wd, np.zeros((4, c_in, 3, 3)), bias, pool=2)
    assert phi0.shape == (n, 4 * 4 * 4) and np.array_equal(phi0.reshape(n, 4, -1), np.broadcast_to(np.maximum(bias, 0)[None, :, None], (n, 4, 16)))
    # a shift tap (reads the pixel to the left) shows the zero padding and the tap orientation: row y, column 0 sees 0
    shift = np.zeros((1, 1, 3, 3)); shift[0, 0, 1, 0] = 1.0
    img = np.arange(16, dtype=np.float32).reshape(1, 16) + 1.0
    got = O.conv_pool_features(img, 1, 4, 4, shift, np.zeros(1), pool=1).reshape(4, 4)
    expect = np.zeros((4, 4)); expect[:, 1:] = (img.reshape(4, 4))[:, :-1]
    assert np.array_equal(got, expect)
    # general case against torch in float64 (signed inputs, bias, rectifier, 2 x 2 pooling), bf16 storage widened exactly
    xt = torch.randn((5, 3, 8, 8), dtype=torch.float32, generator=torch.Generator().manual_seed(32)).to(torch.bfloat16)
    wt = torch.randn((6, 3, 3, 3), dtype=torch.float64, generator=torch.Generator().manual_seed(33)) * 0.4
    bt = torch.randn((6,), dtype=torch.float64, generator=torch.Generator().manual_seed(34)) * 0.2
    ref = torch.nn.functional.avg_pool2d(torch.relu(torch.nn.functional.conv2d(xt.double(), wt, bt, padding=1)), 2).reshape(5, -1).numpy()
    bits = xt.reshape(5, -1).view(torch.int16).numpy().view(np.uint16)
    mine = O.conv_pool_features(bits, 3, 8, 8, wt.numpy(), bt.numpy(), pool=2)
    assert np.allclose(mine, ref, rtol=1e-13, atol=1e-13)
    # 5 x 5 taps use padding 2
    w5 = torch.randn((2, 3, 5, 5), dtype=torch.float64, generator=torch.Generator().manual_seed(35)) * 0.2
    ref5 = torch.nn.functional.avg_pool2d(torch.relu(torch.nn.functional.conv2d(xt.double(), w5, None, padding=2)), 4).reshape(5, -1).numpy()
    assert np.allclose(O.conv_pool_features(bits, 3, 8, 8, w5.numpy(), np.zeros(2), pool=4), ref5, rtol=1e-13, atol=1e-13)


def test_bf16_rounding_is_nearest_even():
    src = np.array([1.0, 1.00390625, 1.01171875, -3.0e-41, 3.3895314e38, np.inf], np.float32)
    ref = torch.from_numpy(src).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.round_bf16(src), ref)
    rnd = np.random.default_rng(16).standard_normal(10000).astype(np.float32)
    ref = torch.from_numpy(rnd).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(O.round_bf16(rnd), ref)


def test_composed_mlp_step_descends_the_objective_to_first_order():
    """assistant_step_mlp chains score_mlp, labels, mlp_grad, sgd and round_bf16: one small step from parameters whose
    W1 is exactly representable in bf16 must lower the mean cross-entropy by lr * |grad|^2 to first order, with the
    gradient taken by central differences of the objective (not by the oracle's own backward pass)."""
    rng = np.random.default_rng(5)
    n, d, hidden = 40, 6, 5
    x = rng.normal(size=(n, d)).astype(np.float32)
    W1 = (rng.integers(-32, 32, size=(hidden, d)) / 16.0).astype(np.float32)        # bf16-exact values
    W1_bits = O.round_bf16(W1)
    b1 = rng.normal(size=hidden).astype(np.float32) * 0.3
    w2 = rng.normal(size=hidden).astype(np.float32)
    b2 = np.float32(0.2)
    f = np.abs(rng.normal(size=n)).astype(np.float32)
    T = float(np.median(f))
    z = O.labels(f, T)

    def objective(theta):
        W1_, b1_, w2_, b2_ = theta[:hidden * d].reshape(hidden, d), theta[hidden * d:hidden * d + hidden], \
            theta[hidden * d + hidden:hidden * d + 2 * hidden], theta[-1]
        return O.bce_mean(O.score_mlp(x, W1_, b1_, w2_, b2_), z)

    theta0 = np.concatenate([W1.reshape(-1), b1, w2, [b2]]).astype(np.float64)
    probe = theta0.copy()
    g_fd = _fd(lambda: objective(probe), probe)
    lr = 1e-3
    out = O.assistant_step_mlp(x, f, W1, W1_bits, b1, w2, b2, lr, T=T)
    theta1 = np.concatenate([out["W1"].reshape(-1), out["b1"], out["w2"], [out["b2"]]]).astype(np.float64)
    # the update is -lr times the finite-difference gradient (fp32 rounding of the parameters aside)
    assert np.allclose(theta0 - theta1, lr * g_fd, rtol=2e-3, atol=2e-7)
    drop = objective(theta0) - objective(theta1)
    assert drop > 0 and abs(drop - lr * float(g_fd @ g_fd)) <= 0.02 * lr * float(g_fd @ g_fd)
    assert np.array_equal(out["W1_bf16"], O.round_bf16(out["W1"]))
    assert np.array_equal(out["z"], z)


def test_mlp_step_with_given_scores_and_the_grad_w2_identity():
    """(1) Handing assistant_step_mlp its own pre-activations changes nothing; handing it other ones changes r only:
    with s = +/- large the residual is 1 - z or -z and grad b2 has the closed form (count of z = 0) / M resp. -(count of z = 1) / M.
    (2) relu(a) = [a > 0] (W1 . x + b1) ties the oracle's four gradients together:
    w2_u grad_w2_u ... = sum_k W1_uk gW1_uk + b1_u gb1_u  (both sides are w2_u sum_i r_i relu(a_iu) / M)."""
    rng = np.random.default_rng(12)
    n, d, hidden = 60, 7, 6
    x = rng.normal(size=(n, d)).astype(np.float32)
    W1 = (rng.integers(-32, 32, size=(hidden, d)) / 16.0).astype(np.float32)
    W1_bits = O.round_bf16(W1)
    b1 = (rng.normal(size=hidden) * 0.3).astype(np.float32)
    w2 = rng.normal(size=hidden).astype(np.float32)
    b2 = np.float32(-0.1)
    f = np.abs(rng.normal(size=n)).astype(np.float32)
    base = O.assistant_step_mlp(x, f, W1, W1_bits, b1, w2, b2, 0.1)
    same = O.assistant_step_mlp(x, f, W1, W1_bits, b1, w2, b2, 0.1, s=base["s"])
    for key in ("W1", "b1", "w2", "b2"):
        assert np.array_equal(np.asarray(base[key]), np.asarray(same[key]))
    z = base["z"]
    hi = O.assistant_step_mlp(x, f, W1, W1_bits, b1, w2, b2, 0.1, s=np.full(n, 60.0))
    lo = O.assistant_step_mlp(x, f, W1, W1_bits, b1, w2, b2, 0.1, s=np.full(n, -60.0))
    assert abs(hi["grads"][3] - float(np.sum(z == 0)) / n) < 1e-12
    assert abs(lo["grads"][3] + float(np.sum(z == 1)) / n) < 1e-12
    gW1, gb1, gw2, gb2 = base["grads"]
    lhs = w2.astype(np.float64) * gw2
    rhs = np.sum(W1.astype(np.float64) * gW1, axis=1) + b1.astype(np.float64) * gb1
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-14)
    assert np.abs(lhs).max() > 1e-3


def test_batch_cut_is_the_literal_walk_of_algorithm_1():
    """batch_cut on the ordered survivors equals the sequential Algorithm 1 loop (batch and candidates consumed), and the
    token-budget form has the closed forms of unit lengths and of a budget nothing fits in."""
    rng = np.random.default_rng(9)
    n = 5000
    g = rng.uniform(0.05, 0.95, n)
    keep = O.shrink(g, 0.1, 4, 2)
    Bfull = O.compact(keep)
    for bs in (1, 7, 64, len(Bfull), len(Bfull) + 10):
        Bseq, consumed_seq = O.sample_batch(g, 0.1, 4, 2, bs)
        b, consumed, _ = O.batch_cut(Bfull, n, batch_size=bs)
        assert b == len(Bseq) and np.array_equal(Bfull[:b], Bseq) and consumed == consumed_seq
    ones = np.ones(n, np.int32)
    b, consumed, off = O.batch_cut(Bfull, n, lengths=ones, token_budget=100)
    assert b == 100 and consumed == Bfull[99] + 1 and np.array_equal(off, np.arange(101))
    b, consumed, off = O.batch_cut(Bfull, n, lengths=ones * 5, token_budget=4)
    assert (b, consumed, list(off)) == (0, 0, [0])
    b, consumed, off = O.batch_cut(Bfull, n, lengths=ones, token_budget=10 ** 9)
    assert b == len(Bfull) and consumed == n and off[-1] == len(Bfull)
    lengths = rng.integers(8, 129, n).astype(np.int32)
    b, consumed, off = O.batch_cut(Bfull, n, lengths=lengths, token_budget=25000, batch_size=300)
    assert b == 300 and off[-1] == lengths[Bfull[:300]].sum() <= 25000      # the instance limit binds first here
    b, consumed, off = O.batch_cut(Bfull, n, lengths=lengths, token_budget=2500)
    assert off[-1] <= 2500 < off[-1] + lengths[Bfull[b]] and np.array_equal(np.diff(off), lengths[Bfull[:b]])


def test_hard_shrinking_rule():
    v = np.array([0.0, 0.5, 0.5000001, 0.4999999, np.nan, np.inf, -1.0, 2.0], np.float32)
    keep = O.hard_shrink(v, 0.5)
    assert list(keep) == [0, 1, 1, 0, 0, 1, 0, 1]                  # >= keeps, NaN drops
    rng = np.random.default_rng(3)
    v = rng.exponential(1.0, 20000).astype(np.float32)
    counts = [int(O.hard_shrink(v, T).sum()) for T in (0.0, 0.5, 1.0, 2.0, 50.0)]
    assert counts[0] == v.size and counts[-1] == 0 and all(a >= b for a, b in zip(counts, counts[1:]))
    assert abs(counts[2] / v.size - math.exp(-1.0)) < 0.01          # P(Exp(1) >= 1) = 1/e
    assert np.array_equal(O.compact(O.hard_shrink(v, 1.0)), np.nonzero(v >= np.float32(1.0))[0])
    assert O.sk_threshold(3.0, 1) == 3.0 and math.isclose(O.sk_threshold(3.0, 12), 0.25, rel_tol=1e-6)


def test_adam_rule_matches_torch_and_closed_forms():
    import torch

    rng = np.random.default_rng(21)
    p0 = rng.normal(size=37).astype(np.float32)
    grads = [rng.normal(size=37) * 0.1 for _ in range(5)]
    # library routine: torch.optim.Adam in float64 on the same gradients
    tp = torch.tensor(p0.astype(np.float64), requires_grad=True)
    opt = torch.optim.Adam([tp], lr=0.01, betas=(0.9, 0.999), eps=1e-8)
    p, m, v = p0.copy(), np.zeros(37, np.float32), np.zeros(37, np.float32)
    for t, g in enumerate(grads, 1):
        tp.grad = torch.tensor(g)
        opt.step()
        p, m, v = O.adam(p, m, v, g, 0.01, 0.9, 0.999, 1e-8, t)
        assert np.allclose(p, tp.detach().numpy(), rtol=2e-6, atol=2e-7)
    # first step from zero moments: every coordinate moves by lr * g / (|g| + eps), i.e. lr * sign(g)
    p1, m1, v1 = O.adam(np.zeros(4, np.float32), np.zeros(4, np.float32), np.zeros(4, np.float32),
                        np.array([0.3, -2.0, 1e-3, -1e-3]), 0.05, 0.9, 0.999, 1e-12, 1)
    assert np.allclose(p1, [-0.05, 0.05, -0.05, 0.05], rtol=1e-6)
    assert np.allclose(m1, 0.1 * np.array([0.3, -2.0, 1e-3, -1e-3]), rtol=1e-6) and np.allclose(v1, 1e-3 * np.array([0.09, 4.0, 1e-6, 1e-6]), rtol=1e-4, atol=0)
    # zero gradient with a live first moment still moves the parameter
    p2, _, _ = O.adam(np.zeros(1, np.float32), np.array([0.5], np.float32), np.array([0.25], np.float32), np.zeros(1), 0.1, 0.9, 0.999, 1e-8, 3)
    assert p2[0] < 0


def _pipeline_inputs(n_steps, n=300, d=12, classes=5, seed=31):
    rng = np.random.default_rng(seed)
    pools = [rng.normal(size=(n, d)).astype(np.float32) for _ in range(n_steps)]
    logits = [rng.normal(size=(n, classes)).astype(np.float32) * 2 for _ in range(n_steps)]
    labels = [rng.integers(0, classes, n).astype(np.int32) for _ in range(n_steps)]
    w0 = (rng.normal(size=d) * 0.3).astype(np.float32)
    return pools, logits, labels, w0


def test_pipeline_schedule_lag_and_special_cases():
    """Sec. "Asynchronous joint learning with CPU/GPU" / Algorithms 2-3 as one event sequence: batch j is screened with the parameters after
    max(0, j - depth) updates; depth 0 is the plain chain screen -> loss -> update; a zero learning rate makes the
    depth irrelevant; batches screened before the first update do not depend on the learning rate."""
    steps = 7
    pools, logits, labels, w0 = _pipeline_inputs(steps)
    pool_of = lambda j: pools[j]
    logits_of = lambda j: (logits[j], labels[j])
    runs = {}
    for depth in (0, 1, 3, 10):
        out, lag = O.pipeline_linear_dense(pool_of, logits_of, w0, 0.05, 0.2, 77, 0.5, depth, steps)
        assert lag == [max(0, j - depth) for j in range(steps)]
        runs[depth] = out
        # batch j against a screening with the snapshot the lag names (snapshots come from the run itself)
        snaps = [(w0, np.float32(0.05))] + [(o["w"], o["b"]) for o in out]
        for j in range(steps):
            wj, bj = snaps[lag[j]]
            assert np.array_equal(out[j]["B"], O.screen_linear_dense(pools[j], wj, bj, 0.2, 77, j)["B"])
    # depth 0 == the chain written out by hand
    w, b = w0.copy(), np.float32(0.05)
    for t in range(steps):
        Bt = O.screen_linear_dense(pools[t], w, b, 0.2, 77, t)["B"]
        f = O.row_loss(logits[t][: len(Bt)], labels[t][: len(Bt)])
        w, b, _ = O.assistant_step_linear_dense(pools[t], f, w, b, 0.5, row_idx=Bt.astype(np.int32))
        assert np.array_equal(Bt, runs[0][t]["B"]) and np.array_equal(w, runs[0][t]["w"]) and b == runs[0][t]["b"]
    # a learning rate that moves the parameters makes stale screening visible: some later batch differs between depths
    assert any(not np.array_equal(runs[0][t]["B"], runs[3][t]["B"]) for t in range(1, steps))
    # the first depth+1 batches are screened before any update: identical to depth 10 (all screened with the initial parameters)
    for t in range(4):
        assert np.array_equal(runs[3][t]["B"], runs[10][t]["B"])
    # lr = 0: every depth gives the same batches, and the parameters never move
    base, _ = O.pipeline_linear_dense(pool_of, logits_of, w0, 0.05, 0.2, 77, 0.0, 0, steps)
    for depth in (1, 4):
        other, _ = O.pipeline_linear_dense(pool_of, logits_of, w0, 0.05, 0.2, 77, 0.0, depth, steps)
        for t in range(steps):
            assert np.array_equal(base[t]["B"], other[t]["B"]) and np.array_equal(other[t]["w"], w0)


def test_instance_loss_rows_is_the_row_loss_of_the_listed_rows():
    """Brute force with scipy's logsumexp on the listed rows; the identity list gives the plain per-row losses;
    a repeated entry repeats its loss."""
    from scipy.special import logsumexp

    rng = np.random.default_rng(17)
    lg = (rng.normal(size=(50, 9)) * 3).astype(np.float32)
    y = rng.integers(0, 9, 50).astype(np.int32)
    rows = np.array([49, 0, 7, 7, 23, 1], np.int32)
    got = O.instance_loss_rows(lg, y, rows)
    want = [logsumexp(lg[r].astype(np.float64)) - float(lg[r, y[r]]) for r in rows]
    assert np.allclose(got, want, rtol=1e-12, atol=1e-12)
    assert got[2] == got[3]
    assert np.array_equal(O.instance_loss_rows(lg, y, np.arange(50)), O.row_loss(lg, y))
