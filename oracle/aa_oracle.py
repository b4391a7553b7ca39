"""NumPy front end of the CPU oracle (test infrastructure, not the product).

Builds ``aa_oracle.c`` with gcc on first use and exposes each of its functions
on NumPy arrays.  fp32 parameters are widened to fp64 here (exactly) because
the oracle carries everything in fp64.  bf16 data travels as ``uint16`` bit
patterns.  Nothing in this module touches CUDA or the product package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aa_oracle.c")
_LIB = os.path.join(_HERE, "libaa_oracle.so")

F32, BF16 = 0, 1

_c_i64 = ctypes.c_int64
_c_u64 = ctypes.c_uint64
_c_dbl = ctypes.c_double
_vp = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the oracle (-O2, no fast-math) if the library is missing or stale."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fno-fast-math", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.aa_ref_uniform.restype = _c_dbl
        _lib.aa_ref_uniform.argtypes = [_c_u64, _c_u64, _c_u64]
        _lib.aa_ref_shrink.restype = _c_i64
        _lib.aa_ref_compact.restype = _c_i64
        _lib.aa_ref_sample_batch.restype = _c_i64
        _lib.aa_ref_batch_mean.restype = _c_dbl
        _lib.aa_ref_bce_mean.restype = _c_dbl
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(_vp)


def _arr(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def _data(x):
    """(contiguous array, dtype code) for fp32 or bf16-as-uint16 storage."""
    if x.dtype == np.uint16:
        return np.ascontiguousarray(x), BF16
    if x.dtype == np.float32:
        return np.ascontiguousarray(x), F32
    raise TypeError(f"oracle data must be float32 or uint16 (bf16 bits), got {x.dtype}")


def philox4x32_10(ctr, key) -> np.ndarray:
    ctr = _arr(ctr, np.uint32)
    key = _arr(key, np.uint32)
    out = np.zeros(4, dtype=np.uint32)
    lib().aa_ref_philox4x32_10(_p(ctr), _p(key), _p(out))
    return out


def uniform(seed: int, step: int, ids) -> np.ndarray:
    f = lib().aa_ref_uniform
    return np.array([f(seed, step, int(i)) for i in np.atleast_1d(ids)], dtype=np.float64)


def score_dense(x, w, b, row_idx=None, n_cand=None) -> np.ndarray:
    x, dt = _data(x)
    row_idx = _arr(row_idx, np.int32)
    n = int(n_cand if n_cand is not None else (len(row_idx) if row_idx is not None else x.shape[0]))
    w = _arr(w, np.float64)
    s = np.zeros(n, dtype=np.float64)
    lib().aa_ref_score_dense(_p(x), dt, _c_i64(x.shape[1]), _c_i64(x.shape[1]), _p(row_idx),
                             _c_i64(n), _p(w), _c_dbl(float(b)), _p(s))
    return s


def score_csr(indptr, col, val, w, b, row_idx=None, n_cand=None) -> np.ndarray:
    indptr, col, val = _arr(indptr, np.int32), _arr(col, np.int32), _arr(val, np.float32)
    row_idx = _arr(row_idx, np.int32)
    n = int(n_cand if n_cand is not None else (len(row_idx) if row_idx is not None else len(indptr) - 1))
    w = _arr(w, np.float64)
    s = np.zeros(n, dtype=np.float64)
    lib().aa_ref_score_csr(_p(indptr), _p(col), _p(val), _p(row_idx), _c_i64(n), _p(w),
                           _c_dbl(float(b)), _p(s))
    return s


def score_mlp(x, W1, b1, w2, b2, row_idx=None, n_cand=None, want_pre=False):
    """W1 is [hidden, d] (fp64 values of whatever precision the caller stores)."""
    x, dt = _data(x)
    row_idx = _arr(row_idx, np.int32)
    n = int(n_cand if n_cand is not None else (len(row_idx) if row_idx is not None else x.shape[0]))
    W1 = _arr(W1, np.float64)
    hidden, d = W1.shape
    assert d == x.shape[1]
    b1, w2 = _arr(b1, np.float64), _arr(w2, np.float64)
    s = np.zeros(n, dtype=np.float64)
    a = np.zeros((n, hidden), dtype=np.float64) if want_pre else None
    lib().aa_ref_score_mlp(_p(x), dt, _c_i64(d), _c_i64(d), _p(row_idx), _c_i64(n), _c_i64(hidden),
                           _p(W1), _p(b1), _p(w2), _c_dbl(float(b2)), _p(s), _p(a))
    return (s, a) if want_pre else s


def sigmoid(s) -> np.ndarray:
    s = _arr(s, np.float64)
    g = np.zeros_like(s)
    lib().aa_ref_sigmoid(_p(s), _c_i64(s.size), _p(g))
    return g


def accept_prob(g, gamma: float) -> np.ndarray:
    g = _arr(g, np.float64)
    p = np.zeros_like(g)
    lib().aa_ref_accept_prob(_p(g), _c_i64(g.size), _c_dbl(gamma), _p(p))
    return p


def shrink(g, gamma: float, seed: int, step: int, id_base: int = 0, row_idx=None) -> np.ndarray:
    g = _arr(g, np.float64)
    row_idx = _arr(row_idx, np.int32)
    keep = np.zeros(g.size, dtype=np.uint8)
    m = lib().aa_ref_shrink(_p(g), _c_i64(g.size), _c_dbl(gamma), _c_u64(seed), _c_u64(step),
                            _c_i64(id_base), _p(row_idx), _p(keep))
    assert m == int(keep.sum())
    return keep


def compact(keep, row_idx=None) -> np.ndarray:
    keep = _arr(keep, np.uint8)
    row_idx = _arr(row_idx, np.int32)
    B = np.zeros(keep.size, dtype=np.int32)
    m = lib().aa_ref_compact(_p(keep), _c_i64(keep.size), _p(row_idx), _p(B))
    return B[:m].copy()


def sample_batch(g, gamma: float, seed: int, step: int, batch_size: int, id_base: int = 0, row_idx=None):
    """Algorithm 1 run literally; returns (B, candidates consumed)."""
    g = _arr(g, np.float64)
    row_idx = _arr(row_idx, np.int32)
    B = np.zeros(max(batch_size, 1), dtype=np.int32)
    consumed = _c_i64(0)
    m = lib().aa_ref_sample_batch(_p(g), _c_i64(g.size), _c_dbl(gamma), _c_u64(seed), _c_u64(step),
                                  _c_i64(id_base), _p(row_idx), _c_i64(batch_size), _p(B),
                                  ctypes.byref(consumed))
    return B[:m].copy(), int(consumed.value)


def row_loss(logits, labels) -> np.ndarray:
    logits, dt = _data(logits)
    labels = _arr(labels, np.int32)
    rows, cols = logits.shape
    ell = np.zeros(rows, dtype=np.float64)
    lib().aa_ref_row_loss(_p(logits), dt, _c_i64(rows), _c_i64(cols), _c_i64(cols), _p(labels), _p(ell))
    return ell


def segment_sum(ell, offsets) -> np.ndarray:
    ell = _arr(ell, np.float64)
    offsets = _arr(offsets, np.int32)
    L = np.zeros(len(offsets) - 1, dtype=np.float64)
    lib().aa_ref_segment_sum(_p(ell), _p(offsets), _c_i64(L.size), _p(L))
    return L


def instance_loss(logits, labels, offsets=None) -> np.ndarray:
    ell = row_loss(logits, labels)
    return ell if offsets is None else segment_sum(ell, offsets)


def batch_mean(f) -> float:
    f = _arr(f, np.float32)
    return float(lib().aa_ref_batch_mean(_p(f), _c_i64(f.size)))


def labels(f, T: float) -> np.ndarray:
    f = _arr(f, np.float32)
    z = np.zeros(f.size, dtype=np.uint8)
    lib().aa_ref_labels(_p(f), _c_i64(f.size), _c_dbl(T), _p(z))
    return z


def bce_mean(s, z) -> float:
    s = _arr(s, np.float64)
    z = _arr(z, np.uint8)
    return float(lib().aa_ref_bce_mean(_p(s), _p(z), _c_i64(s.size)))


def linear_grad_dense(x, s, z, row_idx=None):
    x, dt = _data(x)
    s, z = _arr(s, np.float64), _arr(z, np.uint8)
    row_idx = _arr(row_idx, np.int32)
    d = x.shape[1]
    gw = np.zeros(d, dtype=np.float64)
    gb = _c_dbl(0.0)
    lib().aa_ref_linear_grad_dense(_p(x), dt, _c_i64(d), _c_i64(d), _p(row_idx), _c_i64(s.size),
                                   _p(s), _p(z), _p(gw), ctypes.byref(gb))
    return gw, float(gb.value)


def linear_grad_csr(indptr, col, val, d: int, s, z, row_idx=None):
    indptr, col, val = _arr(indptr, np.int32), _arr(col, np.int32), _arr(val, np.float32)
    s, z = _arr(s, np.float64), _arr(z, np.uint8)
    row_idx = _arr(row_idx, np.int32)
    gw = np.zeros(d, dtype=np.float64)
    gb = _c_dbl(0.0)
    lib().aa_ref_linear_grad_csr(_p(indptr), _p(col), _p(val), _c_i64(d), _p(row_idx), _c_i64(s.size),
                                 _p(s), _p(z), _p(gw), ctypes.byref(gb))
    return gw, float(gb.value)


def mlp_grad(x, a, s, z, w2, row_idx=None):
    x, dt = _data(x)
    a, s, z, w2 = _arr(a, np.float64), _arr(s, np.float64), _arr(z, np.uint8), _arr(w2, np.float64)
    row_idx = _arr(row_idx, np.int32)
    m, hidden = a.shape
    d = x.shape[1]
    gW1 = np.zeros((hidden, d), dtype=np.float64)
    gb1 = np.zeros(hidden, dtype=np.float64)
    gw2 = np.zeros(hidden, dtype=np.float64)
    gb2 = _c_dbl(0.0)
    lib().aa_ref_mlp_grad(_p(x), dt, _c_i64(d), _c_i64(d), _p(row_idx), _c_i64(m), _c_i64(hidden),
                          _p(a), _p(s), _p(z), _p(w2), _p(gW1), _p(gb1), _p(gw2), ctypes.byref(gb2))
    return gW1, gb1, gw2, float(gb2.value)


def conv_pool_features(x, c_in: int, height: int, width: int, weight, bias, pool: int) -> np.ndarray:
    """Features of the convolutional Assistant: phi [n, c_out * (height // pool) * (width // pool)] in fp64.

    x: [n, c_in * height * width] rows (fp32 or bf16 bits), channel-major images; weight [c_out, c_in, k, k], bias [c_out].
    """
    x, dt = _data(x)
    weight = _arr(weight, np.float64)
    bias = _arr(bias, np.float64)
    c_out, ci, k, k2 = weight.shape
    assert ci == c_in and k == k2 and k % 2 == 1 and height % pool == 0 and width % pool == 0
    assert x.shape[1] == c_in * height * width
    n = x.shape[0]
    F = c_out * (height // pool) * (width // pool)
    phi = np.zeros((n, F), dtype=np.float64)
    lib().aa_ref_conv_pool_features(_p(x), dt, _c_i64(x.shape[1]), _c_i64(n), _c_i64(c_in), _c_i64(height), _c_i64(width),
                                    _c_i64(c_out), _c_i64(k), _c_i64(pool), _p(weight), _p(bias), _p(phi))
    return phi


def sgd(param, grad, lr: float) -> np.ndarray:
    """Returns the updated fp32 parameters (input is not modified)."""
    out = np.array(param, dtype=np.float32, copy=True).reshape(-1)
    grad = _arr(np.asarray(grad).reshape(-1), np.float64)
    assert out.size == grad.size
    lib().aa_ref_sgd(_p(out), _c_i64(out.size), _p(grad), _c_dbl(lr))
    return out.reshape(np.shape(param))


def round_bf16(src) -> np.ndarray:
    src = _arr(src, np.float32)
    dst = np.zeros(src.shape, dtype=np.uint16)
    lib().aa_ref_round_bf16(_p(src), _c_i64(src.size), _p(dst))
    return dst


# ---- whole steps, composed from the functions above in the paper's order ----

def screen_linear_dense(x, w, b, gamma, seed, step, id_base=0, row_idx=None):
    """Score -> g -> Bernoulli shrink -> ordered batch B.  Returns dict of every stage."""
    s = score_dense(x, w, b, row_idx=row_idx)
    g = sigmoid(s)
    keep = shrink(g, gamma, seed, step, id_base, row_idx)
    return {"s": s, "g": g, "p": accept_prob(g, gamma), "keep": keep, "B": compact(keep, row_idx)}


def assistant_step_linear_dense(x, f, w, b, lr, T=None, row_idx=None, s=None):
    """Labels from losses f, gradient under the current (w, b), one SGD update.

    T=None uses the batch mean of f.  s: optional pre-activations of the batch instances that the caller already
    holds for these parameters (what screening computed, Algorithm 1); None evaluates them here.
    Returns (w_new fp32, b_new fp32, z).
    """
    f = _arr(f, np.float32)
    if f.size == 0:
        return np.array(w, np.float32, copy=True), np.float32(b), np.zeros(0, np.uint8)
    T = batch_mean(f) if T is None else float(T)
    z = labels(f, T)
    s = score_dense(x, w, b, row_idx=row_idx, n_cand=f.size) if s is None else _arr(s, np.float64)
    gw, gb = linear_grad_dense(x, s, z, row_idx=row_idx)
    w_new = sgd(w, gw, lr)
    b_new = sgd(np.array([b], np.float32), np.array([gb]), lr)[0]
    return w_new, b_new, z


def assistant_step_linear_csr(indptr, col, val, f, w, b, lr, T=None, row_idx=None):
    f = _arr(f, np.float32)
    if f.size == 0:
        return np.array(w, np.float32, copy=True), np.float32(b), np.zeros(0, np.uint8)
    T = batch_mean(f) if T is None else float(T)
    z = labels(f, T)
    s = score_csr(indptr, col, val, w, b, row_idx=row_idx, n_cand=f.size)
    gw, gb = linear_grad_csr(indptr, col, val, len(w), s, z, row_idx=row_idx)
    w_new = sgd(w, gw, lr)
    b_new = sgd(np.array([b], np.float32), np.array([gb]), lr)[0]
    return w_new, b_new, z


def assistant_step_mlp(x, f, W1, W1_bf16, b1, w2, b2, lr, T=None, row_idx=None, s=None):
    """Two-layer Assistant: labels from losses f, back-propagation under the current parameters, one SGD update.

    s: optional pre-activations of the batch instances that the caller already holds for these parameters (what
    screening computed, Algorithm 1); the hidden pre-activations a are evaluated here either way.

    The forward pass reads the bf16 copy of W1 (uint16 bit patterns, as scoring does); the update goes to the fp32
    master, which is then rounded to nearest even into the new bf16 copy.
    Returns dict(W1, W1_bf16, b1, w2, b2, z, grads=(gW1, gb1, gw2, gb2), a, s).
    """
    f = _arr(f, np.float32)
    W1_vals = (np.ascontiguousarray(W1_bf16, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    T = batch_mean(f) if T is None else float(T)
    z = labels(f, T)
    s_here, a = score_mlp(x, W1_vals, b1, w2, b2, row_idx=row_idx, n_cand=f.size, want_pre=True)
    s = s_here if s is None else _arr(s, np.float64)
    gW1, gb1, gw2, gb2 = mlp_grad(x, a, s, z, w2, row_idx=row_idx)
    W1_new = sgd(W1, gW1, lr)
    return {
        "W1": W1_new, "W1_bf16": round_bf16(W1_new), "b1": sgd(b1, gb1, lr), "w2": sgd(w2, gw2, lr),
        "b2": sgd(np.array([b2], np.float32), np.array([gb2]), lr)[0], "z": z, "grads": (gW1, gb1, gw2, gb2), "a": a, "s": s,
    }


def batch_cut(B, n_cand: int, batch_size: int = 0, lengths=None, token_budget: int = 0):
    """The batch Algorithm 1 returns, cut from the ordered survivors B, written as the literal walk: take survivors in
    order until the batch holds batch_size of them (0 = no limit) or, with sentence lengths, until the next one would
    push the token total past token_budget.  Returns (b, consumed, offsets): consumed = position right after the last
    instance taken when a limit ended the walk, n_cand when the survivors ran out; offsets = running token totals."""
    B = np.asarray(B, dtype=np.int64)
    b, tokens, offsets, limited = 0, 0, [0], False
    for r in B:
        if batch_size > 0 and b == batch_size:
            limited = True
            break
        if lengths is not None:
            ln = max(int(lengths[r]), 0)
            if tokens + ln > token_budget:
                limited = True
                break
            tokens += ln
            offsets.append(tokens)
        b += 1
    if batch_size > 0 and b == batch_size:
        limited = True
    consumed = (int(B[b - 1]) + 1 if b > 0 else 0) if limited else int(n_cand)
    return b, consumed, np.asarray(offsets, dtype=np.int64)


def hard_shrink(value, T: float) -> np.ndarray:
    """Hard shrinking (Eq. "shrinking_grad"): instance i is used iff its objective value / gradient magnitude is >= T."""
    value = np.asarray(value, dtype=np.float32)
    keep = np.zeros(value.size, dtype=np.uint8)
    for i in range(value.size):
        keep[i] = 1 if float(value[i]) >= float(np.float32(T)) else 0
    return keep


def sk_threshold(G: float, k: int) -> float:
    """Threshold schedule of the convergence theorem: T_k = G / k."""
    return float(np.float32(G) / np.float32(k))


def adam(param, m, v, grad, lr: float, beta1: float, beta2: float, eps: float, t: int):
    """One Adam update (Kingma & Ba; the optimizer the paper's Assistants were trained with), elementwise in fp64 on
    fp32 state: returns (param, m, v) rounded once to fp32.  t = number of this step, starting at 1."""
    p64 = np.asarray(param, np.float32).astype(np.float64)
    m64 = np.asarray(m, np.float32).astype(np.float64)
    v64 = np.asarray(v, np.float32).astype(np.float64)
    g64 = np.asarray(grad, np.float64).reshape(p64.shape)
    b1, b2 = float(np.float32(beta1)), float(np.float32(beta2))
    m_new = np.empty_like(m64); v_new = np.empty_like(v64); p_new = np.empty_like(p64)
    for j in np.ndindex(p64.shape):
        m_new[j] = b1 * m64[j] + (1.0 - b1) * g64[j]
        v_new[j] = b2 * v64[j] + (1.0 - b2) * g64[j] * g64[j]
        m_hat = m_new[j] / (1.0 - b1 ** t)
        v_hat = v_new[j] / (1.0 - b2 ** t)
        p_new[j] = p64[j] - lr * m_hat / (np.sqrt(v_hat) + float(np.float32(eps)))
    return p_new.astype(np.float32), m_new.astype(np.float32), v_new.astype(np.float32)


def pipeline_linear_dense(pool_of, logits_of, w, b, gamma: float, seed: int, lr: float, depth: int, n_steps: int, T=None):
    """The Assistant / Boss schedule of Sec. "Asynchronous joint learning with CPU/GPU" (Algorithms 2 and 3) with a Boss queue of `depth` batches, written
    as the one sequence of events it becomes when both workers take turns in a fixed order:

      Assistant: while the Boss queue is short (fewer than `depth` batches ahead of the Boss, and always the batch the
                 Boss needs next), screen the next pool with the CURRENT parameters and enqueue its batch;
      Boss:      pop batch t, evaluate its per-instance losses, push (batch, losses) to the Assistant queue;
      Assistant: pop that item, take one update.

    So batch j is screened with the parameters after max(0, j - depth) updates; depth = 0 is the sequential path.
    pool_of(j) -> feature matrix of pool j (bf16 bits or fp32); logits_of(j) -> (logits, labels) whose row i belongs
    to the i-th instance of batch j.  Batch j is screened with Philox step j.
    Returns a list of per-step dicts {B, f, w, b} (w, b = parameters after that step's update) and the list `lag`
    with lag[j] = number of updates the parameters had seen when batch j was screened.
    """
    w_cur = np.array(w, np.float32, copy=True)
    b_cur = np.float32(b)
    queue = {}
    lag = []
    updates = 0
    next_screen = 0
    out = []
    for t in range(n_steps):
        # Assistant: sampling has priority over updating while the Boss queue is short
        while next_screen < n_steps and next_screen <= t + depth:
            r = screen_linear_dense(pool_of(next_screen), w_cur, b_cur, gamma, seed, next_screen)
            queue[next_screen] = r["B"]
            lag.append(updates)
            next_screen += 1
        # Boss: losses of batch t
        Bt = queue.pop(t)
        lg, lab = logits_of(t)
        f = instance_loss(lg[: len(Bt)], np.asarray(lab)[: len(Bt)])
        # Assistant: one update on (batch t, losses)
        w_cur, b_cur, _ = assistant_step_linear_dense(pool_of(t), f, w_cur, b_cur, lr, T=T, row_idx=np.asarray(Bt, np.int32))
        updates += 1
        out.append({"B": Bt, "f": f, "w": w_cur.copy(), "b": np.float32(b_cur)})
    return out, lag


def instance_loss_rows(logits, labels, row_idx) -> np.ndarray:
    """Losses of the batch instances (Sec. "Asynchronous joint learning with CPU/GPU": {f(x_i, y_i)} for i in B) out of logits / labels stored for the whole
    pool: entry k is the row loss of stored row row_idx[k]."""
    labels = _arr(labels, np.int32)
    out = np.zeros(len(row_idx), dtype=np.float64)
    for k, r in enumerate(np.asarray(row_idx, dtype=np.int64)):
        out[k] = row_loss(logits[r: r + 1], labels[r: r + 1])[0]
    return out
